"""Parity of the CUDA path (through the C ABI) with the CPU oracle on the same seeded inputs.

Bars (written here, used below):
  * coreset indices in fp64 deterministic mode: identical ordered lists;
  * attend on the ORACLE's coreset: max_j ||gpu_j - ref_j||_inf / ||ref_j||_inf
      <= 1e-4 for fp32 inputs, <= 2e-2 for bf16 inputs (fp32 mode), <= 2e-6 / 1e-2 in fp64 mode
      (the output is still rounded to the storage type);
  * end-to-end error against exact attention within 1.05 x the oracle's (mean over seeds);
  * fp32 mode indices: structure valid, mismatch rate reported (printed).
"""
import numpy as np
import pytest
import torch

import paper_2606_10944_b200 as elm
from paper_2606_10944_b200.workloads import WORKLOADS, generate

from _util import (check_coreset_structure, e_fro, e_max, max_rel_err, mismatch_rate,
                   oracle_attend, oracle_compress, oracle_exact)

pytestmark = pytest.mark.gpu

ATTEND_TOL = {("f32", "fp32"): 1e-4, ("bf16", "fp32"): 2e-2, ("f32", "fp64"): 2e-6, ("bf16", "fp64"): 1e-2}


def _dev(*ts):
    return [t.cuda() if t is not None else None for t in ts]


def _compress_both(wl, seed=1, data_seed=1234, precision="fp64", delta_level=None):
    _, K, V = generate(wl, seed=data_seed, want_q=False)
    Kd, Vd = _dev(K, V)
    idx, w = elm.compress(Kd, Vd, wl.log2_nout, wl.m, seed=seed, precision=precision, delta_level=delta_level)
    torch.cuda.synchronize()
    ref_idx, ref_w, margins = oracle_compress(K, V, wl.log2_nout, wl.m, seed=seed, delta_level=delta_level)
    return idx.cpu().numpy(), w.cpu().numpy(), ref_idx, ref_w, margins


def _assert_bit_exact(idx, ref_idx, margins):
    if not np.array_equal(idx, ref_idx):
        bad = np.argwhere(idx != ref_idx)[0]
        raise AssertionError(f"first index mismatch at {tuple(bad)}: gpu {idx[tuple(bad)]} oracle "
                             f"{ref_idx[tuple(bad)]}; oracle min margin |U-p| = {margins.min():.3e}")


# ----------------------------------------------------------------------------------------------
# compress, fp64 deterministic mode: ordered index lists identical to the oracle's
# ----------------------------------------------------------------------------------------------
SMALL_CASES = {
    # several tiles and ragged structure: calls smaller than a warp, equal to it, and spanning tiles
    "cfg1_full": WORKLOADS["cfg1"],
    "cfg2_two_batches": WORKLOADS["cfg2"].scaled(batch=2, q_heads=3, kv_heads=3),
    "cfg3_four_heads": WORKLOADS["cfg3"].scaled(batch=2, q_heads=2, kv_heads=2),
    "cfg4_n8192": WORKLOADS["cfg4"].scaled(q_heads=2, kv_heads=2, n=8192, n_q=8192),
    "cfg5_n8192": WORKLOADS["cfg5"].scaled(q_heads=4, kv_heads=2, n=8192, n_q=8192),
    "cfg5_n2048_g4": WORKLOADS["cfg5"].scaled(q_heads=2, kv_heads=2, n=2048, n_q=64, g=4),
    "mixture_d128_f32": WORKLOADS["cfg2"].scaled(batch=1, q_heads=2, kv_heads=2, n=4096, d=128, g=1),
    "lowrank_d64_bf16": WORKLOADS["cfg3"].scaled(batch=1, q_heads=4, kv_heads=2, n=4096, n_q=700, d=64, g=1),
}


@pytest.mark.parametrize("name", sorted(SMALL_CASES))
def test_compress_fp64_indices_identical(name):
    wl = SMALL_CASES[name]
    idx, w, ref_idx, ref_w, margins = _compress_both(wl)
    _assert_bit_exact(idx, ref_idx, margins)
    assert np.array_equal(w, ref_w.astype(np.float32))
    assert np.allclose(w.sum(-1), 1.0, atol=1e-6) and (w > 0).all()
    check_coreset_structure(idx, wl.n, wl.m)


@pytest.mark.parametrize("log2_nout,m,d,dtype", [
    (6, 0, 64, "f32"),      # m = 0: nothing is thinned
    (5, 1, 64, "bf16"),     # one Halve call over everything
    (1, 2, 64, "f32"),      # smallest legal groups: 2 points per level-0 call
    (2, 3, 128, "bf16"),
    (4, 5, 64, "f32"),      # group sizes 2, 4, ..., 32
    (7, 2, 128, "f32"),
    (9, 1, 64, "bf16"),     # one call with 512 pairs: many 32-pair blocks in one walk
])
def test_compress_fp64_edge_shapes(log2_nout, m, d, dtype):
    n = (1 << log2_nout) << m
    wl = WORKLOADS["cfg2"].scaled(batch=1, q_heads=2, kv_heads=2, n=n, n_q=8, d=d, dtype=dtype)
    _, K, V = generate(wl, seed=7, want_q=False)
    Kd, Vd = _dev(K, V)
    idx, w = elm.compress(Kd, Vd, log2_nout, m, seed=3, precision="fp64")
    ref_idx, ref_w, margins = oracle_compress(K, V, log2_nout, m, seed=3)
    _assert_bit_exact(idx.cpu().numpy(), ref_idx, margins)
    assert np.array_equal(w.cpu().numpy(), ref_w.astype(np.float32))


def test_compress_fp64_custom_delta_levels_and_seed_dependence():
    wl = WORKLOADS["cfg2"].scaled(batch=1, q_heads=1, kv_heads=1)
    dl = [0.5, 0.5, 0.5]
    a = _compress_both(wl, seed=11, delta_level=dl)
    _assert_bit_exact(a[0], a[2], a[4])
    b = _compress_both(wl, seed=12, delta_level=dl)
    _assert_bit_exact(b[0], b[2], b[4])
    assert not np.array_equal(a[0], b[0])
    c = _compress_both(wl, seed=11)                    # default schedule differs from constant 1/2
    _assert_bit_exact(c[0], c[2], c[4])
    big = _compress_both(wl, seed=(5 << 32) + 11, delta_level=dl)   # high seed word is used
    _assert_bit_exact(big[0], big[2], big[4])
    assert not np.array_equal(a[0], big[0])


def test_compress_degenerate_inputs():
    """Identical points (a_i = 0 everywhere) and huge keys (shifted exponents far below the floor)."""
    n, d = 256, 64
    K = torch.ones(1, 1, n, d) * 0.25
    V = torch.ones(1, 1, n, d)
    idx, _ = elm.compress(K.cuda(), V.cuda(), 5, 3, seed=2, precision="fp64")
    ref_idx, _, mg = oracle_compress(K, V, 5, 3, seed=2)
    _assert_bit_exact(idx.cpu().numpy(), ref_idx, mg)
    g = torch.Generator().manual_seed(5)
    K = torch.randn(1, 2, n, d, generator=g) * 6.0
    K[0, 0, 100] *= 4.0
    V = torch.randn(1, 2, n, d, generator=g)
    idx, _ = elm.compress(K.cuda(), V.cuda(), 5, 3, seed=2, precision="fp64")
    ref_idx, _, mg = oracle_compress(K, V, 5, 3, seed=2)
    _assert_bit_exact(idx.cpu().numpy(), ref_idx, mg)


# full-size problems of the two largest workloads (one / two KV heads of the real shape)
@pytest.mark.parametrize("name,heads", [("cfg4", 2), ("cfg5", 2)])
def test_compress_fp64_full_size_heads(name, heads):
    wl = WORKLOADS[name].scaled(q_heads=heads, kv_heads=heads, n_q=8)
    idx, w, ref_idx, ref_w, margins = _compress_both(wl)
    _assert_bit_exact(idx, ref_idx, margins)
    check_coreset_structure(idx, wl.n, wl.m)


# ----------------------------------------------------------------------------------------------
# compress, fp32 mode: valid structure, mismatch rate reported
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("name", ["cfg1_full", "cfg2_two_batches", "cfg3_four_heads", "cfg5_n8192", "cfg4_n8192",
                                  "lowrank_d64_bf16"])
def test_compress_fp32_structure_and_mismatch_rate(name):
    wl = SMALL_CASES[name]
    idx, w, ref_idx, ref_w, _ = _compress_both(wl, precision="fp32")
    check_coreset_structure(idx, wl.n, wl.m)
    assert np.allclose(w, 1.0 / wl.n_out)
    rate = mismatch_rate(idx, ref_idx)
    print(f"[fp32 mode] {name}: index mismatch rate vs fp64 oracle = {rate:.4f}")
    assert rate < 0.5          # an unrelated coreset of this structure would mismatch ~ 1 - 2^-m


# ----------------------------------------------------------------------------------------------
# attend on the oracle's coreset
# ----------------------------------------------------------------------------------------------
def _attend_case(wl, precision, weights="uniform", n_core=None, data_seed=99):
    Q, K, V = generate(wl, seed=data_seed)
    rng = np.random.default_rng(data_seed)
    if n_core is None:
        ref_idx, ref_w, _ = oracle_compress(K, V, wl.log2_nout, wl.m, seed=4)
    else:
        ref_idx = np.stack([[rng.permutation(wl.n)[:n_core] for _ in range(wl.kv_heads)]
                            for _ in range(wl.batch)]).astype(np.int32)
        ref_w = np.full(ref_idx.shape, 1.0 / n_core)
    if weights == "random":
        ref_w = (rng.random(ref_idx.shape) + 0.05).astype(np.float32).astype(np.float64)
    Qd, Kd, Vd = _dev(Q, K, V)
    O = elm.attend(Qd, Kd, Vd, torch.from_numpy(ref_idx).cuda(),
                   torch.from_numpy(ref_w.astype(np.float32)).cuda(), precision=precision)
    ref = oracle_attend(Q, K, V, ref_idx, ref_w.astype(np.float32).astype(np.float64))
    err = max_rel_err(O.float().cpu().numpy(), ref)
    return err, ATTEND_TOL[(wl.dtype, precision)]


@pytest.mark.parametrize("precision", ["fp32", "fp64"])
@pytest.mark.parametrize("name", ["cfg1_full", "cfg2_two_batches", "cfg3_four_heads", "cfg5_n8192", "lowrank_d64_bf16"])
def test_attend_on_oracle_coreset(name, precision):
    wl = SMALL_CASES[name]
    wl = wl.scaled(n_q=min(wl.n_q, 1000))            # ragged last query tile
    err, tol = _attend_case(wl, precision)
    print(f"[attend {precision}] {name}: max rel err {err:.3e} (bar {tol:g})")
    assert err <= tol


@pytest.mark.parametrize("dtype,d,n_core,n_q,hq,hkv", [
    ("f32", 64, 1, 5, 2, 2), ("f32", 64, 33, 70, 4, 2), ("bf16", 128, 100, 129, 4, 1),
    ("bf16", 64, 257, 64, 2, 2), ("f32", 128, 512, 31, 6, 3), ("bf16", 128, 2048, 300, 8, 2),
])
def test_attend_arbitrary_weights_and_ragged_shapes(dtype, d, n_core, n_q, hq, hkv):
    wl = WORKLOADS["cfg2"].scaled(batch=2, q_heads=hq, kv_heads=hkv, n=4096, n_q=n_q, d=d, dtype=dtype)
    for precision in ("fp32", "fp64"):
        err, tol = _attend_case(wl, precision, weights="random", n_core=n_core)
        assert err <= tol, (precision, err)


@pytest.mark.parametrize("dtype,d,n_core,n_q,hq,hkv", [
    ("bf16", 128, 2048, 1, 8, 2),     # decode: one new token, 4 query heads per KV head
    ("bf16", 128, 12288, 1, 4, 4),    # a full Express cache (6 n_out entries), no grouping
    ("f32", 64, 301, 2, 4, 1),        # 8 query vectors per KV head, ragged list
    ("bf16", 64, 1, 3, 2, 2),         # single entry
    ("f32", 128, 70, 1, 1, 1),        # list shorter than one CTA's share
    ("bf16", 128, 4096, 5, 8, 8),     # 5 rows per head (odd count, padded to 8 vectors)
])
def test_attend_few_queries_takes_the_decode_kernels(dtype, d, n_core, n_q, hq, hkv):
    """(q_heads / kv_heads) * n_q <= 8 in fp32 mode: the HBM-bound decode kernels, same tolerances."""
    wl = WORKLOADS["cfg2"].scaled(batch=2, q_heads=hq, kv_heads=hkv, n=16384, n_q=n_q, d=d, dtype=dtype)
    before = elm.launch_count()
    err, tol = _attend_case(wl, "fp32", weights="random", n_core=n_core)
    assert elm.launch_count() - before == 2          # partial + merge: no gather launch
    assert err <= tol, err


def test_attend_weight_scale_invariance_and_single_point():
    wl = WORKLOADS["cfg2"].scaled(batch=1, q_heads=2, kv_heads=2, n=1024, n_q=100)
    Q, K, V = generate(wl, seed=5)
    Qd, Kd, Vd = _dev(Q, K, V)
    idx = torch.arange(0, 1024, 8, dtype=torch.int32).repeat(1, 2, 1).cuda()
    w = torch.rand(1, 2, 128, generator=torch.Generator().manual_seed(0)).cuda() + 0.1
    a = elm.attend(Qd, Kd, Vd, idx, w, precision="fp64")
    b = elm.attend(Qd, Kd, Vd, idx, w * 1024.0, precision="fp64")
    # the weights enter as an fp32 logit bias log2(w): a scale changes its rounding (~1e-6 relative)
    assert torch.allclose(a, b, rtol=2e-5, atol=2e-6)
    one = elm.attend(Qd, Kd, Vd, idx[..., 5:6].contiguous(), w[..., 5:6].contiguous(), precision="fp32")
    assert torch.allclose(one, Vd[:, :, 40:41, :].expand_as(one), rtol=1e-6, atol=1e-7)


# ----------------------------------------------------------------------------------------------
# end to end against exact attention
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("name", ["cfg2_two_batches", "cfg3_four_heads"])
def test_end_to_end_error_within_5_percent_of_oracle(name):
    wl = SMALL_CASES[name].scaled(n_q=256)
    Q, K, V = generate(wl, seed=77)
    Qd, Kd, Vd = _dev(Q, K, V)
    exact = oracle_exact(Q, K, V)
    gpu_e, ora_e, gpu_f, ora_f = [], [], [], []
    for seed in range(8):
        idx, w = elm.compress(Kd, Vd, wl.log2_nout, wl.m, seed=seed, precision="fp32")
        O = elm.attend(Qd, Kd, Vd, idx, w, precision="fp32").float().cpu().numpy()
        ref_idx, ref_w, _ = oracle_compress(K, V, wl.log2_nout, wl.m, seed=seed)
        Oo = oracle_attend(Q, K, V, ref_idx, ref_w)
        gpu_e.append(e_max(O, exact)); ora_e.append(e_max(Oo, exact))
        gpu_f.append(e_fro(O, exact)); ora_f.append(e_fro(Oo, exact))
    print(f"[e2e] {name}: E_max gpu {np.mean(gpu_e):.4e} oracle {np.mean(ora_e):.4e}; "
          f"E_F gpu {np.mean(gpu_f):.4e} oracle {np.mean(ora_f):.4e}")
    assert np.mean(gpu_e) <= 1.05 * np.mean(ora_e)
    assert np.mean(gpu_f) <= 1.05 * np.mean(ora_f)


def test_full_pipeline_fp64_equals_oracle_pipeline():
    wl = SMALL_CASES["cfg2_two_batches"].scaled(n_q=128)
    Q, K, V = generate(wl, seed=3)
    Qd, Kd, Vd = _dev(Q, K, V)
    idx, w = elm.compress(Kd, Vd, wl.log2_nout, wl.m, seed=9, precision="fp64")
    O = elm.attend(Qd, Kd, Vd, idx, w, precision="fp64").cpu().numpy()
    ref_idx, ref_w, _ = oracle_compress(K, V, wl.log2_nout, wl.m, seed=9)
    assert np.array_equal(idx.cpu().numpy(), ref_idx)
    assert max_rel_err(O, oracle_attend(Q, K, V, ref_idx, ref_w)) <= 2e-6


def test_host_call_matches_device_calls():
    wl = SMALL_CASES["cfg3_four_heads"].scaled(n_q=512)
    Q, K, V = generate(wl, seed=8)
    O, idx, w = elm.compress_attend_host(Q, K, V, wl.log2_nout, wl.m, seed=6, want_coreset=True)
    Qd, Kd, Vd = _dev(Q, K, V)
    idx_d, w_d = elm.compress(Kd, Vd, wl.log2_nout, wl.m, seed=6)
    O_d = elm.attend(Qd, Kd, Vd, idx_d, w_d)
    assert torch.equal(idx, idx_d.cpu()) and torch.equal(w, w_d.cpu()) and torch.equal(O, O_d.cpu())


def test_launch_counter_and_stage_profile():
    wl = SMALL_CASES["cfg2_two_batches"]
    Q, K, V = generate(wl, seed=8)
    Qd, Kd, Vd = _dev(Q, K, V)
    before = elm.launch_count()
    elm.profile_enable(True)
    idx, w = elm.compress(Kd, Vd, wl.log2_nout, wl.m)
    elm.attend(Qd, Kd, Vd, idx, w)
    prof = elm.profile_read()
    elm.profile_enable(False)
    launched = elm.launch_count() - before
    assert launched == sum(v[1] for v in prof.values()) and launched >= 3 * wl.m + 3
    assert prof["attend"][0] > 0 and prof["walk"][1] == wl.m


def test_stage_profile_of_the_attention_stage_only():
    """elm_profile_enable(2): events around the attention stage alone, launches counted for every stage, and the
    results of the step are those of an unprofiled one (the compression's launches then keep their device-side
    ordering without events between them)."""
    wl = SMALL_CASES["cfg3_four_heads"]
    Q, K, V = generate(wl, seed=8)
    Qd, Kd, Vd = _dev(Q, K, V)
    idx0, w0 = elm.compress(Kd, Vd, wl.log2_nout, wl.m, seed=4)
    O0 = elm.attend(Qd, Kd, Vd, idx0, w0)
    elm.profile_enable(2)
    idx, w = elm.compress(Kd, Vd, wl.log2_nout, wl.m, seed=4)
    O = elm.attend(Qd, Kd, Vd, idx, w)
    prof = elm.profile_read()
    elm.profile_enable(False)
    assert prof["attend"][0] > 0 and prof["attend"][1] >= 1
    for stage in ("prepass", "level_prep", "gram", "walk", "emit"):
        assert prof[stage][0] == 0.0 and prof[stage][1] >= 1
    assert torch.equal(idx, idx0) and torch.equal(w, w0) and torch.equal(O, O0)
