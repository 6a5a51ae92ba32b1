"""Pins for the CPU oracle: everything here runs without a GPU.

The oracle is checked against things other than itself: published Philox vectors, NumPy /
SciPy statements of the definitions (matrix form of the kernel, of the pair Gram and of
softmax), brute force over all swap patterns on tiny inputs, the streaming form of
Compress2, and the structural facts the paper states.
"""
import math
import os

import numpy as np
import pytest
from scipy.special import softmax

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _data(seed, n, d, kscale=1.0):
    rng = np.random.default_rng(seed)
    K = (rng.standard_normal((n, d)) * kscale).astype(np.float32)
    V = rng.standard_normal((n, d)).astype(np.float32)
    return K, V


def _gram(K, V, vmax):
    """Eq. (katt) as one matrix expression (float64)."""
    K = K.astype(np.float64)
    V = V.astype(np.float64)
    d = K.shape[1]
    return np.exp(K @ K.T / math.sqrt(d)) * (V @ V.T + vmax * vmax)


def _pair_gram(G):
    """F = P G P^T with P the +1/-1 pairing matrix: F[j,i] = <f_j, f_i> in the RKHS."""
    s = G.shape[0]
    P = np.zeros((s // 2, s))
    P[np.arange(s // 2), 2 * np.arange(s // 2)] = 1.0
    P[np.arange(s // 2), 2 * np.arange(s // 2) + 1] = -1.0
    return P @ G @ P.T


# --------------------------------------------------------------------------------------
# generator
# --------------------------------------------------------------------------------------
def test_philox_known_answers():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        v = [int(x, 16) for x in r]
        out = oracle.philox4x32_10(v[0:4], v[4:6])
        assert [int(x) for x in out] == v[6:10]


def test_uniform_is_24_bit_and_uses_all_counters():
    seen = set()
    for pair, group, level, head in [(0, 0, 0, 0), (1, 0, 0, 0), (0, 1, 0, 0), (0, 0, 1, 0), (0, 0, 0, 1)]:
        u = oracle.uniform(7, pair, group, level, head)
        assert 0.0 <= u < 1.0
        assert u * 2 ** 24 == int(u * 2 ** 24)           # multiple of 2^-24
        assert np.float32(u) == u                        # exact in fp32
        seen.add(u)
    assert len(seen) == 5
    assert oracle.uniform(7, 3, 2, 1, 0) != oracle.uniform(8, 3, 2, 1, 0)
    assert oracle.uniform(7, 3, 2, 1, 0) != oracle.uniform(7 + (1 << 32), 3, 2, 1, 0)
    # first word of the block, top 24 bits
    w = oracle.philox4x32_10([3, 2, 1, 0], [7, 0])
    assert oracle.uniform(7, 3, 2, 1, 0) == (int(w[0]) >> 8) / 2 ** 24
    us = np.array([oracle.uniform(1, i, 0, 0, 0) for i in range(20000)])
    assert abs(us.mean() - 0.5) < 0.01 and abs((us < 0.25).mean() - 0.25) < 0.01


# --------------------------------------------------------------------------------------
# kernel
# --------------------------------------------------------------------------------------
def test_katt_matches_matrix_definition():
    K, V = _data(0, 12, 5)
    vm = oracle.vmax(V)
    assert vm == np.abs(V).max()
    G = _gram(K, V, vm)
    for a in range(12):
        for b in range(12):
            assert oracle.katt(K, V, vm, a, b) == pytest.approx(G[a, b], rel=1e-13)
    # shift multiplies by exp(-shift); the floor zeroes tiny exponents only
    assert oracle.katt(K, V, vm, 1, 2, shift=3.0) == pytest.approx(G[1, 2] * math.exp(-3.0), rel=1e-13)
    assert oracle.katt(K, V, vm, 1, 2, shift=900.0, use_floor=True) == 0.0
    assert oracle.katt(K, V, vm, 1, 2, shift=3.0, use_floor=True) == oracle.katt(K, V, vm, 1, 2, shift=3.0)


def test_katt_is_symmetric_psd():
    K, V = _data(1, 16, 4)
    vm = oracle.vmax(V)
    G = np.array([[oracle.katt(K, V, vm, a, b) for b in range(16)] for a in range(16)])
    assert np.allclose(G, G.T, rtol=1e-14)
    assert np.linalg.eigvalsh(G).min() > -1e-9 * np.abs(G).max()


# --------------------------------------------------------------------------------------
# KH (Algorithm A.1)
# --------------------------------------------------------------------------------------
def _check_against_matrix_form(K, V, x, delta, U, S1, S2, diag, rel=1e-9):
    """Recompute alpha_i, a_i, p_i from F = P G P^T and the decisions actually taken."""
    vm = oracle.vmax(V)
    s = len(x)
    G = _gram(K[x], V[x], vm)
    F = _pair_gram(G)
    eta = np.where(diag[:, 3] > 0.5, -1.0, 1.0)          # +1: x_{2i-1} stayed in S1
    b = np.sqrt(np.clip(np.diag(F), 0, None))
    bmax = np.maximum.accumulate(b)
    a = b * bmax * (0.5 + math.log(2 * s / delta))
    for i in range(s // 2):
        alpha = -np.dot(eta[:i], F[:i, i])
        scale = np.abs(F[:i, i]).sum() + 1e-300
        assert abs(diag[i, 0] - alpha) <= rel * scale
        assert diag[i, 1] == pytest.approx(a[i], rel=1e-9)
        p = min(1.0, 0.5 * max(0.0, 1.0 - alpha / a[i])) if a[i] > 0 else 0.5
        assert diag[i, 2] == pytest.approx(p, abs=1e-8)
        assert (diag[i, 3] > 0.5) == (U[i] < diag[i, 2])
        pair = {int(x[2 * i]), int(x[2 * i + 1])}
        assert {int(S1[i]), int(S2[i])} == pair            # one point of each pair per side
        assert int(S1[i]) == (int(x[2 * i + 1]) if diag[i, 3] > 0.5 else int(x[2 * i]))


@pytest.mark.parametrize("seed,s,d,shift_mode", [(0, 16, 3, 0), (1, 32, 8, 0), (2, 32, 8, 1), (3, 64, 4, 1)])
def test_kh_matches_pair_gram_form(seed, s, d, shift_mode):
    K, V = _data(seed, s + 7, d, kscale=0.7)
    rng = np.random.default_rng(100 + seed)
    x = rng.permutation(s + 7)[:s].astype(np.int32)       # scattered rows, arbitrary order
    U = rng.random(s // 2)
    S1, S2, diag = oracle.kh(K, V, oracle.vmax(V), x, 0.5, U, shift_mode=shift_mode)
    if shift_mode == 0:
        _check_against_matrix_form(K, V, x, 0.5, U, S1, S2, diag)
    else:
        # shifted run: alpha and a are both scaled by exp(-M_i); the ratio and p are not
        S1u, S2u, diagu = oracle.kh(K, V, oracle.vmax(V), x, 0.5, U, shift_mode=0)
        assert np.array_equal(S1, S1u) and np.array_equal(S2, S2u)
        assert np.allclose(diag[:, 2], diagu[:, 2], atol=1e-10)
        ratio = diag[:, 0] / diag[:, 1]
        ratiou = diagu[:, 0] / diagu[:, 1]
        assert np.allclose(ratio, ratiou, atol=1e-9)
        # the scale actually applied is exp(-prefix max of ||k||^2/sqrt(d))
        c = (K[x].astype(np.float64) ** 2).sum(1) / math.sqrt(d)
        M = np.maximum.accumulate(np.maximum(c[0::2], c[1::2]))
        assert np.allclose(diag[:, 1], diagu[:, 1] * np.exp(-M), rtol=1e-9)


def test_kh_first_pair_is_a_fair_coin():
    K, V = _data(5, 2, 6)
    vm = oracle.vmax(V)
    x = np.array([0, 1], dtype=np.int32)
    S1, _, diag = oracle.kh(K, V, vm, x, 0.5, np.array([0.3]))
    assert diag[0, 0] == 0.0 and diag[0, 2] == 0.5 and S1[0] == 1
    S1, _, diag = oracle.kh(K, V, vm, x, 0.5, np.array([0.5]))
    assert S1[0] == 0                                      # swap iff U < p, strictly
    # empirical frequency over Philox seeds
    swaps = sum(oracle.uniform(seed, 0, 0, 0, 0) < 0.5 for seed in range(4000))
    assert abs(swaps / 4000 - 0.5) < 0.03


def test_kh_identical_pair_gives_half():
    K, V = _data(6, 6, 4)
    K[3] = K[2]
    V[3] = V[2]
    x = np.arange(6, dtype=np.int32)
    _, _, diag = oracle.kh(K, V, oracle.vmax(V), x, 0.5, np.array([0.9, 0.9, 0.9]))
    assert diag[1, 1] == 0.0 and diag[1, 2] == 0.5


def test_kh_brute_force_all_patterns_tiny():
    """s = 8: force each of the 16 swap patterns, check every step against the matrix form,
    and that the pattern probabilities form a distribution."""
    K, V = _data(7, 8, 3, kscale=0.8)
    x = np.arange(8, dtype=np.int32)
    total = 0.0
    for pattern in range(16):
        want = [(pattern >> i) & 1 for i in range(4)]
        U = np.array([0.0 if wnt else 1.0 - 2.0 ** -24 for wnt in want])
        S1, S2, diag = oracle.kh(K, V, oracle.vmax(V), x, 0.5, U, shift_mode=0)
        _check_against_matrix_form(K, V, x, 0.5, U, S1, S2, diag)
        prob = 1.0
        for i in range(4):
            p = diag[i, 2]
            took = diag[i, 3] > 0.5
            if took != bool(want[i]):       # forced choice impossible (p is 0 or 1)
                prob = 0.0
                break
            prob *= p if took else 1.0 - p
        total += prob
    assert total == pytest.approx(1.0, abs=1e-12)


def test_kh_mmd_identity():
    """MMD^2(in, S1) from its definition equals eta^T F eta / s^2."""
    K, V = _data(8, 40, 5, kscale=0.6)
    vm = oracle.vmax(V)
    x = np.arange(40, dtype=np.int32)
    U = np.random.default_rng(3).random(20)
    S1, S2, diag = oracle.kh(K, V, vm, x, 0.5, U)
    w = np.full(20, 1.0 / 20)
    got = oracle.mmd2(K, V, vm, x, S1, w)
    G = _gram(K, V, vm)
    ref = G.mean() - 2 * G[:, S1].mean() + G[np.ix_(S1, S1)].mean()
    assert got == pytest.approx(ref, rel=1e-9, abs=1e-12 * G.max())
    eta = np.where(diag[:, 3] > 0.5, -1.0, 1.0)
    F = _pair_gram(G)
    assert got == pytest.approx(eta @ F @ eta / 40 ** 2, rel=1e-7, abs=1e-12 * G.max())


def test_kh_large_keys_need_the_shift_and_survive_it():
    """Exponents far beyond exp's range: the shifted walk stays finite and well formed."""
    K, V = _data(9, 64, 8, kscale=12.0)          # ||k||^2/sqrt(d) ~ 400..., products overflow fp64
    K[17] *= 3.0                                 # one extreme outlier
    x = np.arange(64, dtype=np.int32)
    U = np.random.default_rng(4).random(32)
    S1, S2, diag = oracle.kh(K, V, oracle.vmax(V), x, 0.5, U)
    assert np.isfinite(diag).all()
    assert ((diag[:, 2] >= 0) & (diag[:, 2] <= 1)).all()
    assert sorted(np.concatenate([S1, S2]).tolist()) == list(range(64))


def test_kh_balances_better_than_uniform_on_one_large_call():
    """One large Halve call (not a benchmark config): kernel halving beats a random half."""
    rng = np.random.default_rng(11)
    s, d = 1024, 2
    K = (rng.standard_normal((s, d)) * 0.8).astype(np.float32)
    V = np.tanh(K @ rng.standard_normal((d, d))).astype(np.float32)
    vm = oracle.vmax(V)
    x = np.arange(s, dtype=np.int32)
    G = _gram(K, V, vm)

    def mmd(sel):
        return math.sqrt(max(G.mean() - 2 * G[:, sel].mean() + G[np.ix_(sel, sel)].mean(), 0.0))

    kh_m, un_m = [], []
    for t in range(4):
        U = rng.random(s // 2)
        S1, _, _ = oracle.kh(K, V, vm, x, 0.5, U)
        kh_m.append(mmd(S1))
        un_m.append(mmd(rng.permutation(s)[: s // 2]))
    assert np.mean(kh_m) < 0.8 * np.mean(un_m)


def test_kh_sub_gaussian_bound_per_test_function():
    """|mean_in f - mean_S1 f| <= nu sqrt(2 log(2/delta')) for f = k(z,.)/sqrt(k(z,z)),
    nu^2 = 4 max_i k(x_i,x_i) log(2 s/delta)/s^2, in at least 1 - delta/2 - delta' of runs."""
    s, d, delta, dprime = 64, 4, 0.5, 0.1
    K, V = _data(12, s, d, kscale=0.6)
    vm = oracle.vmax(V)
    G = _gram(K, V, vm)
    x = np.arange(s, dtype=np.int32)
    nu = math.sqrt(4 * np.diag(G).max() * math.log(2 * s / delta)) / s
    bound = nu * math.sqrt(2 * math.log(2 / dprime))
    z = 5
    f = G[z] / math.sqrt(G[z, z])
    ok = 0
    runs = 200
    for seed in range(runs):
        U = np.array([oracle.uniform(seed, i, 0, 0, 0) for i in range(s // 2)])
        S1, _, _ = oracle.kh(K, V, vm, x, delta, U)
        ok += abs(f.mean() - f[S1].mean()) <= bound
    assert ok / runs >= 1 - delta / 2 - dprime


# --------------------------------------------------------------------------------------
# Compress2
# --------------------------------------------------------------------------------------
def _streaming_compress2(K, V, log2_nout, m, delta_level, seed, head):
    """Algorithm 2 (streaming form), one update per point, Halve = the oracle's KH call with the
    same (pair, call number at that level, level, head) counters."""
    n_out = 1 << log2_nout
    n_in = n_out << m
    vm = oracle.vmax(V)
    S = [[] for _ in range(m + 1)]
    calls = [0] * (m + 1)
    for xrow in range(n_in):
        S[0].append(xrow)
        for i in range(m):
            if len(S[i]) == n_in * 2 ** i // 4 ** (m - 1):
                x = np.array(S[i], dtype=np.int32)
                U = np.array([oracle.uniform(seed, p, calls[i], i, head) for p in range(len(x) // 2)])
                S1, _, _ = oracle.kh(K, V, vm, x, float(delta_level[i]), U)
                calls[i] += 1
                S[i + 1].extend(int(t) for t in S1)
                S[i] = []
    return S, calls


@pytest.mark.parametrize("log2_nout,m", [(2, 1), (2, 2), (3, 3), (4, 2)])
def test_compress2_offline_equals_streaming(log2_nout, m):
    n = (1 << log2_nout) << m
    K, V = _data(20 + m, n, 4, kscale=0.7)
    dl = oracle.default_delta_levels(m, 0.5)
    idx, w, margin = oracle.compress2(K, V, log2_nout, m, delta=0.5, seed=5, head=3)
    S, calls = _streaming_compress2(K, V, log2_nout, m, dl, 5, 3)
    assert all(len(S[i]) == 0 for i in range(m))
    assert S[m] == idx.tolist()
    assert calls[:m] == [4 ** (m - 1 - i) for i in range(m)]
    # wtd_cache weights of Algorithm 2: level m carries 2^(m-m) = 1 before normalisation;
    # Definition 1 normalises to a sum of 1
    assert np.all(w > 0) and w.sum() == pytest.approx(1.0, abs=1e-12)
    assert np.all(w == 1.0 / (1 << log2_nout))
    assert 0.0 <= margin <= 1.0


def test_compress2_group_sizes_from_golden():
    """Algorithm 2's size rule, as stored in the golden file, against the Halve calls the oracle makes
    (level, points in, number of calls at that level read off the oracle's own call record)."""
    rows = [tuple(map(int, l.split())) for l in open(os.path.join(GOLDEN, "structure_facts.txt"))
            if l.strip() and not l.startswith("#")]
    cases = sorted({(r[0], r[1]) for r in rows})
    assert len(cases) >= 3
    for n_out, m in cases:
        n = n_out << m
        K, V = _data(40 + m, n, 2, kscale=0.3)
        idx, w, calls = oracle.compress2_calls(K, V, int(math.log2(n_out)), m, seed=2)
        assert len(idx) == n_out
        seen = {}
        for level, number, size, _ in calls:
            key = (int(level), int(size))
            assert number == seen.get(key, 0)                         # calls of a level numbered in order
            seen[key] = seen.get(key, 0) + 1
        assert len({lv for lv, _ in seen}) == len(seen) == m           # one size per level, m levels
        for r in rows:
            if (r[0], r[1]) == (n_out, m):
                assert seen[(r[2], r[3])] == r[4], r
        # default schedule: every level spends delta / (3 m), the call delta / 3 (Corollary 2's split)
        assert calls[:, 3].sum() == pytest.approx(0.5 / 3, rel=1e-12)


def test_kh_running_shift_rescales_carried_bmax():
    """The running shift: b_max is carried in the scale of the previous pair and must be multiplied by
    exp(-(M_i - M_{i-1}) / 2) (b is a square root of kernel values) when the shift grows.  Directed case:
    pair 1 has the largest b; pair 2 is two near-identical keys of large norm, which raises the shift while
    its own b is tiny; pair 3 is an ordinary pair whose threshold a_3 = b_3 b_max (...) needs pair 1's b in
    pair 3's scale.  The unshifted run (the printed formula) is the reference: same p, same decisions,
    and a_i equal after undoing the scale exp(-M_i)."""
    d = 4
    K = np.zeros((6, d), np.float32)
    V = np.zeros((6, d), np.float32)
    K[0], K[1] = [1.0, 0, 0, 0], [-1.0, 0.3, 0, 0]
    K[2], K[3] = [0, 2.5, 0, 0], [0, 2.5, 1e-4, 0]
    K[4], K[5] = [0.2, 0, 0.1, 0], [0.1, 0, 0.2, 0]
    V[0], V[1] = [1, 0, 0, 0], [-1, 0.5, 0, 0]
    V[2], V[3] = [0.3, 0.3, 0, 0], [0.3, 0.3, 0, 0]
    V[4], V[5] = [0.5, 0.1, 0, 0], [0.4, 0.2, 0, 0]
    x = np.arange(6, dtype=np.int32)
    vm = oracle.vmax(V)
    G = _gram(K, V, vm)
    F = _pair_gram(G)
    b = np.sqrt(np.diag(F))
    assert b[0] > 5 * b[2] > 25 * b[1]                                # pair 1 dominates, pair 2 is tiny
    c = (K.astype(np.float64) ** 2).sum(1) / math.sqrt(d)
    M = np.maximum.accumulate(np.maximum(c[0::2], c[1::2]))
    assert M[1] - M[0] > 2.0 and M[2] == M[1]                         # the shift grows at pair 2 only
    for U in ([0.9, 0.9, 0.9], [0.1, 0.9, 0.55], [0.1, 0.1, 0.65]):
        U = np.array(U)
        S1, S2, diag = oracle.kh(K, V, vm, x, 0.5, U, shift_mode=1)
        S1u, S2u, diagu = oracle.kh(K, V, vm, x, 0.5, U, shift_mode=0)
        _check_against_matrix_form(K, V, x, 0.5, U, S1u, S2u, diagu)
        assert np.array_equal(S1, S1u)
        assert np.abs(diag[:, 2] - diagu[:, 2]).max() < 1e-12
        assert 0.05 < abs(diag[2, 2] - 0.5) < 0.45                    # pair 3's p is neither 1/2 nor clamped
        assert np.allclose(diag[:, 1], diagu[:, 1] * np.exp(-M), rtol=1e-12)
        # a_3 = b_3 * (pair 1's b) * (1/2 + ln(2 s / delta)), all in pair 3's scale
        assert diag[2, 1] == pytest.approx(b[2] * b[0] * np.exp(-M[2]) * (0.5 + math.log(2 * 6 / 0.5)), rel=1e-10)


def test_compress2_structure_and_identity():
    K, V = _data(30, 256, 6, kscale=0.5)
    idx, w, _ = oracle.compress2(K, V, 8, 0)                        # m = 0: unchanged
    assert idx.tolist() == list(range(256))
    idx, w, _ = oracle.compress2(K, V, 4, 4, seed=9)
    assert len(idx) == 16 and len(set(idx.tolist())) == 16
    assert idx.min() >= 0 and idx.max() < 256
    # level-0 groups are contiguous blocks of 256/4^3 = 4 rows, each keeps 2, and so on upward:
    # the survivors of block [16 t, 16 t + 16) occupy output slot t only.
    assert [int(i) // 16 for i in idx] == list(range(16))
    # different seed, different coreset; same seed, same coreset
    idx2, _, _ = oracle.compress2(K, V, 4, 4, seed=10)
    idx3, _, _ = oracle.compress2(K, V, 4, 4, seed=9)
    assert idx2.tolist() != idx.tolist() and idx3.tolist() == idx.tolist()


def test_compress2_batched_equals_single():
    rng = np.random.default_rng(31)
    K = rng.standard_normal((3, 64, 4)).astype(np.float32)
    V = rng.standard_normal((3, 64, 4)).astype(np.float32)
    idx, w, mg = oracle.compress2_batched(K, V, 3, 3, seed=2)
    for p in range(3):
        i1, w1, m1 = oracle.compress2(K[p], V[p], 3, 3, seed=2, head=p)
        assert i1.tolist() == idx[p].tolist() and m1 == mg[p]


def test_default_delta_levels_budget():
    for m in (1, 3, 6):
        dl = oracle.default_delta_levels(m, 0.5)
        assert dl[m - 1] == pytest.approx(0.5 / (3 * m))
        spent = sum(4 ** (m - 1 - i) * dl[i] for i in range(m))    # calls per level x delta_i
        assert spent == pytest.approx(0.5 / 3)


def test_oversampling_map_for_powers_of_four():
    from paper_2606_10944_b200.workloads import WORKLOADS
    for n, g in [(1024, 0), (1024, 2), (4096, 1)]:
        wl = WORKLOADS["cfg1"].scaled(n=n, g=g)
        assert wl.n_out == 2 ** g * int(math.isqrt(n))
        assert wl.n // 4 ** (wl.m - 1) == 4 ** (g + 1)             # level-0 group size
    assert [(WORKLOADS[k].n_out, WORKLOADS[k].m) for k in sorted(WORKLOADS)] == \
        [(32, 5), (128, 3), (256, 5), (1024, 5), (2048, 6)]


# --------------------------------------------------------------------------------------
# attention
# --------------------------------------------------------------------------------------
def _att_data(seed, n, nq, d):
    rng = np.random.default_rng(seed)
    return (rng.standard_normal((nq, d)).astype(np.float32),
            rng.standard_normal((n, d)).astype(np.float32),
            rng.standard_normal((n, d)).astype(np.float32))


def test_exact_attention_matches_softmax_definition():
    Q, K, V = _att_data(40, 50, 9, 8)
    ref = softmax(Q.astype(np.float64) @ K.astype(np.float64).T / math.sqrt(8), axis=1) @ V.astype(np.float64)
    assert np.allclose(oracle.exact_attention(Q, K, V), ref, rtol=1e-12, atol=1e-14)


def test_weighted_attention_properties():
    Q, K, V = _att_data(41, 40, 7, 8)
    n = 40
    allidx = np.arange(n, dtype=np.int32)
    # (i) every point with equal weights is exact attention
    full = oracle.wtd_attention(Q, K, V, allidx, np.full(n, 1.0 / n))
    assert np.allclose(full, oracle.exact_attention(Q, K, V), rtol=1e-12, atol=1e-14)
    # general weights against the explicit ratio of two weighted sums
    rng = np.random.default_rng(1)
    idx = rng.permutation(n)[:11].astype(np.int32)
    w = rng.random(11) + 0.1
    E = np.exp(Q.astype(np.float64) @ K[idx].astype(np.float64).T / math.sqrt(8)) * w
    ref = (E @ V[idx].astype(np.float64)) / E.sum(1, keepdims=True)
    got = oracle.wtd_attention(Q, K, V, idx, w)
    assert np.allclose(got, ref, rtol=1e-12, atol=1e-14)
    # (ii) scaling all weights changes nothing
    assert np.allclose(oracle.wtd_attention(Q, K, V, idx, 37.5 * w), got, rtol=1e-12, atol=1e-14)
    # (iii) duplicating a point is doubling its weight
    idx_dup = np.concatenate([idx, idx[:1]])
    w_dup = np.concatenate([w, w[:1]])
    w_dbl = w.copy()
    w_dbl[0] *= 2
    assert np.allclose(oracle.wtd_attention(Q, K, V, idx_dup, w_dup),
                       oracle.wtd_attention(Q, K, V, idx, w_dbl), rtol=1e-12, atol=1e-14)
    # (iv) a single point returns its value
    one = oracle.wtd_attention(Q, K, V, np.array([4], dtype=np.int32), np.array([0.3]))
    assert np.allclose(one, np.broadcast_to(V[4].astype(np.float64), one.shape), rtol=1e-14)


def test_weighted_attention_batched_grouped_queries():
    rng = np.random.default_rng(42)
    B, Hq, Hkv, n, nq, d, c = 2, 4, 2, 24, 5, 4, 6
    Q = rng.standard_normal((B, Hq, nq, d)).astype(np.float32)
    K = rng.standard_normal((B, Hkv, n, d)).astype(np.float32)
    V = rng.standard_normal((B, Hkv, n, d)).astype(np.float32)
    idx = np.stack([[rng.permutation(n)[:c] for _ in range(Hkv)] for _ in range(B)]).astype(np.int32)
    w = rng.random((B, Hkv, c)) + 0.1
    O = oracle.wtd_attention_batched(Q, K, V, idx, w)
    E = oracle.exact_attention_batched(Q, K, V)
    for b in range(B):
        for h in range(Hq):
            kv = h // (Hq // Hkv)
            assert np.array_equal(O[b, h], oracle.wtd_attention(Q[b, h], K[b, kv], V[b, kv], idx[b, kv], w[b, kv]))
            assert np.array_equal(E[b, h], oracle.exact_attention(Q[b, h], K[b, kv], V[b, kv]))


def test_end_to_end_error_shrinks_with_coreset_size_and_vanishes_at_m0():
    from paper_2606_10944_b200.workloads import WORKLOADS, generate, as_f32_numpy
    errs = []
    for g in (0, 1, 2, 3):
        e = []
        for seed in range(3):
            wl = WORKLOADS["cfg2"].scaled(batch=1, q_heads=1, kv_heads=1, n=256, n_q=64, d=16, g=g)
            Q, K, V = (as_f32_numpy(t)[0, 0] for t in generate(wl, seed=50 + seed))
            idx, w, _ = oracle.compress2(K, V, wl.log2_nout, wl.m, seed=seed)
            e.append(np.abs(oracle.wtd_attention(Q, K, V, idx, w) - oracle.exact_attention(Q, K, V)).max())
        errs.append(np.mean(e))
    assert errs[0] > errs[2] > errs[3]
    wl = WORKLOADS["cfg1"].scaled(n=64, n_q=8, d=8, g=3)          # n_out = 64 = n, m = 0
    assert wl.m == 0
    Q, K, V = (as_f32_numpy(t)[0, 0] for t in generate(wl, seed=1))
    idx, w, _ = oracle.compress2(K, V, wl.log2_nout, 0)
    assert np.allclose(oracle.wtd_attention(Q, K, V, idx, w), oracle.exact_attention(Q, K, V), rtol=1e-12)
