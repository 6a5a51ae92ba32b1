"""Parity of elm_compress_ragged (Algorithm 2 on any sequence length, sink / window rows kept) with
the streaming Compress2 oracle, and of elm_attend on its multi-level weighted cache.

Bars: fp64 deterministic mode - identical ordered index lists, weights equal to float rounding;
fp32 mode - the parts the sizes fix (sinks, window, S_0, level sizes) identical, the rest reported
as a mismatch rate; attention over the cache - the tolerances of the fixed-size path.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2606_10944_b200 as elm
from paper_2606_10944_b200.workloads import WORKLOADS, as_f32_numpy, generate

from _util import max_rel_err, oracle_attend

pytestmark = pytest.mark.gpu


def _oracle_ragged(K, V, log2_nout, m, n_sink, n_window, seed, delta_level=None):
    B, H, n, d = K.shape
    Kf, Vf = as_f32_numpy(K).reshape(B * H, n, d), as_f32_numpy(V).reshape(B * H, n, d)
    out = [oracle.compress2_stream(Kf[p], Vf[p], log2_nout, m, n_sink, n_window, seed=seed, head=p,
                                   delta_level=delta_level) for p in range(B * H)]
    idx = np.stack([o[0] for o in out]).reshape(B, H, -1)
    w = np.stack([o[1] for o in out]).reshape(B, H, -1)
    return idx, w


# name: (base workload, overrides, log2_nout, m, n_sink, n_window)
CASES = {
    # calls of 4, 8, 16 ... pairs, a partly filled top level, leftovers in every level
    "iid_n1000_sinks": ("cfg1", dict(n=1000, kv_heads=2, q_heads=2), 5, 5, 32, 32),
    "iid_n517_window_only": ("cfg1", dict(n=517, batch=2), 4, 5, 0, 9),
    "mixture_n3000_f32": ("cfg2", dict(n=3000, batch=1, kv_heads=3, q_heads=3), 6, 6, 32, 32),
    "lowrank_bf16_d128_n5000": ("cfg3", dict(n=5000, batch=1, kv_heads=2, q_heads=4), 6, 7, 32, 32),
    "mixture_bf16_n20000": ("cfg5", dict(n=20000, kv_heads=2, q_heads=4), 8, 7, 32, 32),
    "nothing_halved": ("cfg1", dict(n=30), 5, 2, 3, 3),
    "only_sinks_and_window": ("cfg1", dict(n=9), 3, 3, 4, 5),
    "depth_zero": ("cfg1", dict(n=14), 3, 0, 4, 4),
    "full_length": ("cfg3", dict(n=4096, batch=1, kv_heads=2, q_heads=2), 7, 5, 0, 0),
}


def _inputs(name):
    base, over, log2_nout, m, n_sink, n_window = CASES[name]
    wl = WORKLOADS[base].scaled(**dict(over, n_q=8))
    Q, K, V = generate(wl, seed=77)
    return wl, Q, K, V, log2_nout, m, n_sink, n_window


@pytest.mark.parametrize("name", sorted(CASES))
def test_ragged_fp64_cache_identical(name):
    wl, _, K, V, log2_nout, m, n_sink, n_window = _inputs(name)
    idx, w = elm.compress_ragged(K.cuda(), V.cuda(), log2_nout, m, n_sink, n_window, seed=5, precision="fp64")
    torch.cuda.synchronize()
    ref_idx, ref_w = _oracle_ragged(K, V, log2_nout, m, n_sink, n_window, seed=5)
    assert idx.shape == ref_idx.shape
    assert np.array_equal(idx.cpu().numpy(), ref_idx)
    assert np.allclose(w.cpu().numpy(), ref_w, rtol=1e-6, atol=0)
    assert abs(float(w.double().sum(-1).mean()) - 1.0) < 1e-5


def test_ragged_full_length_equals_elm_compress():
    wl, _, K, V, log2_nout, m, _, _ = _inputs("full_length")
    a_idx, a_w = elm.compress_ragged(K.cuda(), V.cuda(), log2_nout, m, seed=9, precision="fp64")
    b_idx, b_w = elm.compress(K.cuda(), V.cuda(), log2_nout, m, seed=9, precision="fp64")
    assert torch.equal(a_idx, b_idx)
    assert torch.allclose(a_w, b_w, rtol=1e-6)


@pytest.mark.parametrize("name", ["iid_n1000_sinks", "mixture_n3000_f32", "lowrank_bf16_d128_n5000", "mixture_bf16_n20000"])
def test_ragged_fp32_mode_structure_and_mismatch_rate(name):
    wl, _, K, V, log2_nout, m, n_sink, n_window = _inputs(name)
    idx, w = elm.compress_ragged(K.cuda(), V.cuda(), log2_nout, m, n_sink, n_window, seed=5, precision="fp32")
    idx, w = idx.cpu().numpy(), w.cpu().numpy()
    ref_idx, ref_w = _oracle_ragged(K, V, log2_nout, m, n_sink, n_window, seed=5)
    assert idx.shape == ref_idx.shape
    assert np.allclose(w, ref_w, rtol=1e-6, atol=0)            # the weights depend on the sizes only
    flat, rflat = idx.reshape(-1, idx.shape[-1]), ref_idx.reshape(-1, idx.shape[-1])
    # what no floating-point decision touches: sinks, S_0 (its weight is 1/n, like sinks and window), window
    raw = np.isclose(ref_w.reshape(-1, idx.shape[-1])[0], 1.0 / wl.n, rtol=1e-9)
    assert np.array_equal(flat[:, raw], rflat[:, raw])
    for row in flat:
        assert len(set(row.tolist())) == len(row) and row.min() >= 0 and row.max() < wl.n
    rate = float(np.mean([1.0 - len(set(a.tolist()) & set(b.tolist())) / len(a) for a, b in zip(flat, rflat)]))
    print(f"[fp32 mode] {name}: cache mismatch rate vs fp64 oracle = {rate:.4f}")
    assert rate < 0.25


@pytest.mark.parametrize("name,precision,tol", [
    ("mixture_n3000_f32", "fp32", 1e-4), ("mixture_n3000_f32", "fp64", 2e-6),
    ("lowrank_bf16_d128_n5000", "fp32", 2e-2), ("mixture_bf16_n20000", "fp32", 2e-2)])
def test_attend_over_the_ragged_cache(name, precision, tol):
    """elm_attend on the oracle's multi-level cache (weights 2^i / n over several levels)."""
    base, over, log2_nout, m, n_sink, n_window = CASES[name]
    wl = WORKLOADS[base].scaled(**dict(over, n_q=300))
    Q, K, V = generate(wl, seed=78)
    ref_idx, ref_w = _oracle_ragged(K, V, log2_nout, m, n_sink, n_window, seed=6)
    O = elm.attend(Q.cuda(), K.cuda(), V.cuda(), torch.from_numpy(ref_idx).cuda(),
                   torch.from_numpy(ref_w.astype(np.float32)).cuda(), precision=precision)
    ref = oracle_attend(Q, K, V, ref_idx, ref_w.astype(np.float32).astype(np.float64))
    err = max_rel_err(O.float().cpu().numpy(), ref)
    print(f"[attend over ragged cache] {name} {precision}: max rel err {err:.2e}")
    assert err <= tol


def test_ragged_end_to_end_error_within_5_percent_of_oracle():
    """End to end on a ragged length with sinks and a window: the error against exact attention of the
    CUDA cache equals that of the oracle's cache (same indices in fp64 mode) and is no worse than 1.05 x
    the oracle's in fp32 mode, averaged over seeds."""
    base, over, log2_nout, m, n_sink, n_window = CASES["mixture_n3000_f32"]
    wl = WORKLOADS[base].scaled(**dict(over, n_q=200))
    Q, K, V = generate(wl, seed=79)
    exact = oracle.exact_attention_batched(as_f32_numpy(Q), as_f32_numpy(K), as_f32_numpy(V))
    errs_gpu, errs_ref = [], []
    for seed in range(4):
        idx, w = elm.compress_ragged(K.cuda(), V.cuda(), log2_nout, m, n_sink, n_window, seed=seed, precision="fp32")
        O = elm.attend(Q.cuda(), K.cuda(), V.cuda(), idx.contiguous(), w.contiguous(), precision="fp32")
        ref_idx, ref_w = _oracle_ragged(K, V, log2_nout, m, n_sink, n_window, seed=seed)
        ref_O = oracle_attend(Q, K, V, ref_idx, ref_w)
        errs_gpu.append(np.abs(O.float().cpu().numpy() - exact).max())
        errs_ref.append(np.abs(ref_O - exact).max())
    print(f"[ragged end to end] max-abs error gpu {np.mean(errs_gpu):.4f} oracle {np.mean(errs_ref):.4f}")
    assert np.mean(errs_gpu) <= 1.05 * np.mean(errs_ref) + 1e-6


def test_ragged_rejects_bad_sizes():
    K = torch.zeros((1, 1, 50, 64), device="cuda")
    with pytest.raises(elm.ElmError):
        elm.compress_ragged(K, K, 3, 2)                       # 50 middle rows > n_in = 32
    with pytest.raises(elm.ElmError):
        elm.compress_ragged(K, K, 3, 3, n_sink=30, n_window=30)
    with pytest.raises(elm.ElmError):
        elm.compress_ragged(K, K, 1, 6)                       # level-0 stretches below one pair
