"""8-bit (E4M3) inputs, the paper's "future work" (Conclusion): the CUDA path against the oracle on the SAME rounded
numbers (the oracle takes the exact upcast of the E4M3 values, as it does for bf16).

Tolerances.  Compression: every E4M3 value is a bf16 value and the kernels run on an exact widened copy, so in fp64 mode
the coreset is identical to the oracle's, as for bf16 inputs.  Attention in fp32 mode: S = Q K^T is computed with 8-bit
tensor-core operands; a product of two E4M3 numbers has at most 8 significant bits, so the products and their fp32
accumulation carry the same rounding as in the bf16 path; probabilities and P V are bf16 as there, and O is rounded to
bf16: the bf16 bar of 2e-2 on the maximum relative error applies unchanged (fp64 mode: 1e-2, the rounding of O).
"""
import numpy as np
import pytest
import torch

import paper_2606_10944_b200 as elm
from paper_2606_10944_b200 import binding
from paper_2606_10944_b200.workloads import WORKLOADS, generate

from _util import e_fro, e_max, max_rel_err, mismatch_rate, oracle_attend, oracle_compress, oracle_exact

pytestmark = pytest.mark.gpu

CASES = {
    # low-rank keys and values, two KV heads with two query heads each, coreset of 256 points over two blocks of 128
    "lowrank_n4096": WORKLOADS["cfg3"].scaled(batch=1, q_heads=4, kv_heads=2, n=4096, n_q=1000, dtype="e4m3"),
    # heavy-tailed key norms (clamped to the format's range), grouped queries
    "mixture_t3_n8192": WORKLOADS["cfg5"].scaled(q_heads=4, kv_heads=1, n=8192, n_q=700, dtype="e4m3"),
}


@pytest.mark.parametrize("name", sorted(CASES))
def test_e4m3_compress_fp64_identical_and_fp32_mismatch_rate(name):
    wl = CASES[name]
    Q, K, V = generate(wl, seed=21)
    assert K.dtype == torch.float8_e4m3fn
    ref_idx, ref_w, _ = oracle_compress(K, V, wl.log2_nout, wl.m, seed=4)
    idx, w = elm.compress(K.cuda(), V.cuda(), wl.log2_nout, wl.m, seed=4, precision="fp64")
    assert np.array_equal(idx.cpu().numpy(), ref_idx)
    assert np.allclose(w.cpu().numpy(), ref_w)
    idx32, _ = elm.compress(K.cuda(), V.cuda(), wl.log2_nout, wl.m, seed=4, precision="fp32")
    rate = mismatch_rate(idx32.cpu().numpy(), ref_idx)
    print(f"{name}: fp32-mode index mismatch rate on E4M3 inputs {rate:.4f}")
    assert rate <= 0.25


@pytest.mark.parametrize("precision,tol", [("fp32", 2e-2), ("fp64", 1e-2)])
@pytest.mark.parametrize("name", sorted(CASES))
def test_e4m3_attend_on_oracle_coreset(name, precision, tol):
    wl = CASES[name]
    Q, K, V = generate(wl, seed=22)
    ref_idx, ref_w, _ = oracle_compress(K, V, wl.log2_nout, wl.m, seed=4)
    O = elm.attend(Q.cuda(), K.cuda(), V.cuda(), torch.from_numpy(ref_idx).cuda(),
                   torch.from_numpy(ref_w.astype(np.float32)).cuda(), precision=precision)
    assert O.dtype == torch.bfloat16
    ref = oracle_attend(Q, K, V, ref_idx, ref_w)
    err = max_rel_err(O.float().cpu().numpy(), ref)
    print(f"{name} {precision}: attend on E4M3 inputs, max relative error {err:.3e}")
    assert err <= tol


@pytest.mark.parametrize("n_core,n_q,hq,hkv", [(300, 77, 4, 2), (128, 513, 2, 2), (1, 40, 2, 1), (2049, 300, 8, 2)])
def test_e4m3_attend_arbitrary_weights_and_ragged_shapes(n_core, n_q, hq, hkv):
    wl = WORKLOADS["cfg5"].scaled(batch=2, q_heads=hq, kv_heads=hkv, n=4096, n_q=n_q, dtype="e4m3")
    Q, K, V = generate(wl, seed=23)
    g = torch.Generator().manual_seed(n_core)
    idx = torch.stack([torch.stack([torch.randperm(wl.n, generator=g)[:n_core] for _ in range(hkv)])
                       for _ in range(2)]).to(torch.int32)
    w = torch.rand(2, hkv, n_core, generator=g) * 4 + 0.01
    O = elm.attend(Q.cuda(), K.cuda(), V.cuda(), idx.cuda(), w.cuda(), precision="fp32")
    ref = oracle_attend(Q, K, V, idx.numpy(), w.numpy().astype(np.float64))
    assert max_rel_err(O.float().cpu().numpy(), ref) <= 2e-2


def test_e4m3_end_to_end_error_within_5_percent_of_oracle():
    wl = CASES["lowrank_n4096"]
    ratios_max, ratios_fro = [], []
    Q, K, V = generate(wl, seed=24)
    exact = oracle_exact(Q, K, V)
    Qd, Kd, Vd = Q.cuda(), K.cuda(), V.cuda()
    gm, gf, om, of_ = [], [], [], []
    for seed in range(8):
        ref_idx, ref_w, _ = oracle_compress(K, V, wl.log2_nout, wl.m, seed=seed)
        ref = oracle_attend(Q, K, V, ref_idx, ref_w)
        idx, w = elm.compress(Kd, Vd, wl.log2_nout, wl.m, seed=seed, precision="fp32")
        got = elm.attend(Qd, Kd, Vd, idx, w, precision="fp32").float().cpu().numpy()
        gm.append(e_max(got, exact)); gf.append(e_fro(got, exact))
        om.append(e_max(ref, exact)); of_.append(e_fro(ref, exact))
    print(f"E4M3 end to end: E_max {np.mean(gm):.4e} (oracle {np.mean(om):.4e}), E_F {np.mean(gf):.4e} (oracle {np.mean(of_):.4e})")
    assert np.mean(gm) <= 1.05 * np.mean(om) and np.mean(gf) <= 1.05 * np.mean(of_)


def test_e4m3_is_refused_where_it_is_not_supported():
    wl = WORKLOADS["cfg2"].scaled(batch=1, q_heads=1, kv_heads=1, dtype="e4m3")     # d = 64
    Q, K, V = generate(wl, seed=1)
    with pytest.raises(elm.ElmError):
        elm.compress(K.cuda(), V.cuda(), wl.log2_nout, wl.m)
    wl = WORKLOADS["cfg3"].scaled(batch=1, q_heads=1, kv_heads=1, n=1024, n_q=1024, dtype="e4m3")
    Q, K, V = generate(wl, seed=1)
    with pytest.raises(elm.ElmError):
        elm.express_compress(K.cuda(), V.cuda(), 4, 2)
