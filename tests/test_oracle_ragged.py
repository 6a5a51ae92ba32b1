"""Pins for the streaming Compress2 oracle (Algorithm 2) on sequences of any length, with sink and
window rows kept exactly.

Checked against what the algorithm fixes: the level sizes after n updates (closed form from the
thresholds n_in 2^i / 4^(m-1)), conservation of mass (every Halve call halves the count and doubles
the weight, so the weights always sum to the number of points fed times 2^-m), the prefix property
of a streaming procedure, agreement with the recursive Offline-Compress2 at full length, and a
direct re-run of single Halve calls through the KH(delta) routine.
"""
import numpy as np
import pytest

import oracle


def _kv(seed, n, d, kscale=0.5):
    rng = np.random.default_rng(seed)
    return ((rng.standard_normal((n, d)) * kscale).astype(np.float32),
            rng.standard_normal((n, d)).astype(np.float32))


def _level_sizes(n_mid, n_out, m):
    """Points left in S_0..S_m after n_mid updates: level i makes floor(a_i / thresh_i) calls."""
    sizes, a = [], n_mid
    for i in range(m):
        thresh = (n_out << (m + i)) >> (2 * (m - 1))
        calls = a // thresh
        sizes.append(a - calls * thresh)
        a = calls * (thresh // 2)
    sizes.append(a)
    return sizes


def _split(idx, w, n, n_sink, n_window, sizes):
    """Cut an output into (sinks, [S_0..S_m], window)."""
    parts, at = [], n_sink
    for s in sizes:
        parts.append((idx[at:at + s], w[at:at + s]))
        at += s
    assert at + n_window == len(idx)
    return (idx[:n_sink], w[:n_sink]), parts, (idx[at:], w[at:])


@pytest.mark.parametrize("log2_nout,m", [(3, 1), (3, 2), (4, 3), (3, 4)])
def test_full_length_equals_offline_compress2(log2_nout, m):
    """With n = 2^m n_out and nothing kept aside, Algorithm 2 and its recursive form agree."""
    n = (1 << log2_nout) << m
    K, V = _kv(10 + m, n, 8)
    idx, w = oracle.compress2_stream(K, V, log2_nout, m, seed=7, head=3)
    ridx, rw, _ = oracle.compress2(K, V, log2_nout, m, seed=7, head=3)
    assert np.array_equal(idx, ridx)
    assert np.allclose(w, rw, rtol=1e-15)


@pytest.mark.parametrize("n,log2_nout,m,n_sink,n_window", [
    (500, 4, 5, 0, 0), (500, 4, 5, 32, 32), (120, 3, 4, 5, 0), (64, 3, 3, 0, 0), (63, 3, 3, 0, 9),
    (130, 5, 2, 1, 1), (14, 3, 0, 4, 4), (9, 3, 3, 4, 5), (100, 3, 4, 0, 0)])
def test_level_sizes_weights_and_order(n, log2_nout, m, n_sink, n_window):
    n_out = 1 << log2_nout
    K, V = _kv(n, n, 4)
    idx, w = oracle.compress2_stream(K, V, log2_nout, m, n_sink, n_window, seed=11)
    sizes = _level_sizes(n - n_sink - n_window, n_out, m)
    assert len(idx) == n_sink + n_window + sum(sizes)
    (si, sw), parts, (wi, ww) = _split(idx, w, n, n_sink, n_window, sizes)
    # sinks and window: exactly those rows, the weight of a raw point
    assert list(si) == list(range(n_sink)) and list(wi) == list(range(n - n_window, n))
    assert np.all(sw == 1.0 / n) and np.all(ww == 1.0 / n)
    # level i: weight 2^i / n; S_0 holds the most recent middle rows, in order
    for i, (pi, pw) in enumerate(parts):
        assert np.all(pw == 2.0 ** i / n)
    s0 = sizes[0]
    assert list(parts[0][0]) == list(range(n - n_window - s0, n - n_window))
    # positive weights summing to 1 (Definition 1); every point appears once; the middle levels hold middle rows
    assert abs(w.sum() - 1.0) < 1e-12 and np.all(w > 0)
    assert len(set(idx.tolist())) == len(idx)
    for pi, _ in parts:
        assert np.all((pi >= n_sink) & (pi < n - n_window))
    # calls are made on consecutive stretches: every survivor comes before the rows still waiting in S_0
    for pi, _ in parts[1:]:
        if len(pi) and s0:
            assert pi.max() < n - n_window - s0


def test_prefix_property():
    """A streaming procedure: what has been halved after t updates does not change later.  The
    levels above 0 after n_mid updates equal those after the largest multiple of the level-0
    threshold below it, and the lower levels of a longer run extend it."""
    log2_nout, m, d = 3, 4, 6
    n_out = 1 << log2_nout
    thresh0 = (n_out << m) >> (2 * (m - 1))
    K, V = _kv(5, 100, d)
    full_idx, full_w = oracle.compress2_stream(K, V, log2_nout, m, seed=3)
    sizes = _level_sizes(100, n_out, m)
    _, parts, _ = _split(full_idx, full_w, 100, 0, 0, sizes)
    cut = (100 // thresh0) * thresh0
    # same K, V rows but only the first `cut`: v_max must not change, so keep the largest |v| inside the prefix
    big = np.abs(V).max(axis=1).argmax()
    V2 = V.copy()
    V2[[0, big]] = V2[[big, 0]]
    K2 = K.copy()
    K2[[0, big]] = K2[[big, 0]]
    a_idx, a_w = oracle.compress2_stream(K2, V2, log2_nout, m, seed=3)
    b_idx, b_w = oracle.compress2_stream(K2[:cut], V2[:cut], log2_nout, m, seed=3)
    sa = _level_sizes(100, n_out, m)
    sb = _level_sizes(cut, n_out, m)
    assert sb[0] == 0 and sa[1:] == sb[1:]
    _, pa, _ = _split(a_idx, a_w, 100, 0, 0, sa)
    _, pb, _ = _split(b_idx, b_w, cut, 0, 0, sb)
    for i in range(1, m + 1):
        assert np.array_equal(pa[i][0], pb[i][0])


def test_single_calls_rerun_through_kh():
    """m = 2, n_out = 8: thresholds 8 (level 0) and 16 (level 1).  20 middle rows: two level-0 calls,
    4 rows left in S_0, 8 survivors waiting in S_1.  Each call is KH(delta_0) on 8 consecutive rows
    with the uniforms of counter (pair, call, level 0, head)."""
    log2_nout, m, n_sink, n_window = 3, 2, 2, 3
    n = 25
    K, V = _kv(21, n, 5)
    idx, w = oracle.compress2_stream(K, V, log2_nout, m, n_sink, n_window, delta=0.25, seed=9, head=4)
    sizes = _level_sizes(20, 8, 2)
    assert sizes == [4, 8, 0]
    _, parts, _ = _split(idx, w, n, n_sink, n_window, sizes)
    dl = oracle.default_delta_levels(2, 0.25)
    vm = oracle.vmax(V)
    want = []
    for call in range(2):
        x = np.arange(n_sink + 8 * call, n_sink + 8 * call + 8, dtype=np.int32)
        U = np.array([oracle.uniform(9, a, call, 0, 4) for a in range(4)])
        S1, _, _ = oracle.kh(K, V, vm, x, dl[0], U)
        want += S1.tolist()
    assert parts[1][0].tolist() == want
    # and once S_1 fills (32 middle rows: four level-0 calls, then one level-1 call on their 16 survivors)
    n = 32
    K, V = _kv(22, n, 5)
    idx, w = oracle.compress2_stream(K, V, log2_nout, m, delta=0.25, seed=9, head=4)
    assert len(idx) == 8 and np.all(w == 4.0 / 32)
    vm = oracle.vmax(V)
    s1 = []
    for call in range(4):
        x = np.arange(8 * call, 8 * call + 8, dtype=np.int32)
        U = np.array([oracle.uniform(9, a, call, 0, 4) for a in range(4)])
        s1 += oracle.kh(K, V, vm, x, dl[0], U)[0].tolist()
    U = np.array([oracle.uniform(9, a, 0, 1, 4) for a in range(8)])
    S2, _, _ = oracle.kh(K, V, vm, np.array(s1, dtype=np.int32), dl[1], U)
    assert idx.tolist() == S2.tolist()


def test_rejects_bad_arguments():
    K, V = _kv(1, 50, 4)
    with pytest.raises(ValueError):
        oracle.compress2_stream(K, V, 3, 2)                    # 50 > n_in = 32
    with pytest.raises(ValueError):
        oracle.compress2_stream(K, V, 3, 3, n_sink=30, n_window=30)
    with pytest.raises(ValueError):
        oracle.compress2_stream(K, V, 1, 6)                    # level-0 threshold below one pair


def test_attention_over_ragged_cache_is_exact_when_nothing_was_halved():
    """Fewer middle rows than the level-0 threshold: every row is still there with equal weight, so
    weighted attention over the cache equals exact attention."""
    n, d = 30, 8
    K, V = _kv(8, n, d)
    Q = np.random.default_rng(9).standard_normal((5, d)).astype(np.float32)
    idx, w = oracle.compress2_stream(K, V, 5, 2, n_sink=3, n_window=3)     # threshold 32 > 24
    assert sorted(idx.tolist()) == list(range(n))
    assert np.allclose(oracle.wtd_attention(Q, K, V, idx, w), oracle.exact_attention(Q, K, V), rtol=1e-12, atol=1e-14)
