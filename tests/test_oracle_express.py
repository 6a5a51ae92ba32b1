"""Pins for the streaming Express / Thinformer Express oracle (Algorithms 1-5, Corollary 2).

Checked against what the paper states in closed form: exactness up to 4 n_out tokens (Theorem 3),
the cache-size bound of Theorem 1, the exact query-cost formula of the WtdAttention cost
proposition at the endpoints n = n_out 4^k, the number of Halve calls in the runtime recursion,
and the equivalence of the streaming procedure with the recursive Offline-Express.
"""
import math

import numpy as np
import pytest

import oracle


def _qkv(seed, n, d, kscale=0.5):
    rng = np.random.default_rng(seed)
    return ((rng.standard_normal((n, d)) * kscale).astype(np.float32),
            (rng.standard_normal((n, d)) * kscale).astype(np.float32),
            rng.standard_normal((n, d)).astype(np.float32))


def _m_n(n, n_out):
    return 2 * math.ceil(math.log(n / (4 * n_out), 4) - 1e-12) if n > 4 * n_out else 0


def test_exact_up_to_four_n_out_tokens():
    """Theorem 3: the approximation equals exact causal attention for every n <= 4 n_out."""
    Q, K, V = _qkv(0, 4 * 16 + 40, 8)
    r = oracle.thinformer_express(Q, K, V, log2_nout=4, mbar=2)
    ex = oracle.exact_causal_attention(Q, K, V)
    assert np.allclose(r["O"][:64], ex[:64], rtol=1e-12, atol=1e-14)
    assert list(r["cache_size"][:64]) == list(range(64))         # nothing thinned: all earlier tokens
    assert np.abs(r["O"][64:] - ex[64:]).max() > 1e-6               # afterwards it is an approximation


@pytest.mark.parametrize("log2_nout,mbar,k", [(3, 2, 2), (3, 4, 3), (4, 2, 2), (4, 4, 3)])
def test_query_cost_closed_form_at_endpoints(log2_nout, mbar, k):
    """The proposition's exact count at n = n_out 4^k with m_n <= mbar:
    (4 n_out)(4 n_out + 1)/2 + (7/2 n_out^2 - n_out/2)(2^(m_n+2) - 4) - 3 (m_n/2) n_out^2.
    Its proof counts the input token itself for the first 4 n_out queries (i points for query i) and
    only the cache (j n_out + a_u + sum_l n_out 2^(l-s) d_{u,l}) afterwards; the same convention here."""
    n_out = 1 << log2_nout
    n = n_out * 4 ** k
    m_n = _m_n(n, n_out)
    assert m_n == 2 * (k - 1) and m_n <= mbar
    Q, K, V = _qkv(1, n, 4)
    r = oracle.thinformer_express(Q, K, V, log2_nout, mbar, want_outputs=False)
    cost = int(r["cache_size"].astype(np.int64).sum()) + 4 * n_out
    closed = (4 * n_out) * (4 * n_out + 1) // 2 + (7 * n_out ** 2 - n_out) * (2 ** (m_n + 2) - 4) // 2 \
        - 3 * (m_n // 2) * n_out ** 2
    assert cost == closed
    assert r["cache_size"].max() < 6 * n_out                         # Theorem 1
    # at a round end only the Express coreset is left: n_out points of weight 1
    assert len(r["final_idx"]) == n_out and np.all(r["final_w"] == 1.0)
    assert len(set(r["final_idx"].tolist())) == n_out


def test_cache_bound_and_query_cost_bound_with_subsampling():
    """m_n > mbar: Subsample keeps one point per stratum; cache < 6 n_out; cost <= the third case."""
    log2_nout, mbar = 3, 2
    n_out = 8
    n = n_out * 4 ** 4                                               # rounds m = 0, 2, 4, 6 > mbar
    Q, K, V = _qkv(2, n, 4)
    r = oracle.thinformer_express(Q, K, V, log2_nout, mbar, want_outputs=False)
    assert r["cache_size"].max() < 6 * n_out
    cost = int(r["cache_size"].astype(np.int64).sum()) + 4 * n_out
    assert cost <= (4 * n_out) * (4 * n_out + 1) // 2 + 6 * n_out * (n - 4 * n_out)
    assert len(r["final_idx"]) == n_out


def test_halve_call_count_matches_runtime_recursion():
    """Per round m: three Compress2(q = min(m, mbar)) instances with sum_i 4^(q-1-i) Halve calls
    each, plus the two halvings of the Express coreset."""
    log2_nout, mbar = 3, 2
    n_out = 8
    for k in (1, 2, 3, 4):
        n = n_out * 4 ** k
        Q, K, V = _qkv(3, n, 4)
        r = oracle.thinformer_express(Q, K, V, log2_nout, mbar, want_outputs=False)
        want = 0
        for rnd in range(k):
            q = min(2 * rnd, mbar)
            want += 3 * sum(4 ** (q - 1 - i) for i in range(q)) + 2
        assert r["halve_calls"] == want


def test_weights_of_a_mid_round_cache():
    """Inside a thin phase the cache is [(S_i, 2^(i-q))] + (E, 1)."""
    log2_nout, mbar = 3, 2
    n_out = 8
    n = 4 * n_out + 4 * n_out + 11                  # round m = 2 (32 .. 128), second sibling, 11 tokens in
    Q, K, V = _qkv(4, n, 4)
    r = oracle.thinformer_express(Q, K, V, log2_nout, mbar, want_outputs=False)
    w = r["final_w"]
    assert set(np.unique(w).tolist()) <= {0.25, 0.5, 1.0}
    assert (w == 1.0).sum() == 2 * n_out            # E: n_out from the halve phase + one finished sibling
    # S_0 holds the raw tail: 11 tokens = one full level-0 group of n_out 2^(2-q) = 8 halved to 4 (weight 1/2)
    # plus 3 raw points (weight 1/4)
    assert (w == 0.25).sum() == 3 and (w == 0.5).sum() == 4
    assert sorted(r["final_idx"][w == 0.25].tolist()) == [n - 3, n - 2, n - 1]


def _offline_express(K, V, vmax, x, n_out, mbar, delta, seed, head):
    """Offline-Express written from its recursion with the oracle's KH as Halve; returns the coreset."""
    n_in = len(x)
    if n_in <= n_out:
        return list(x)
    m = int(round(math.log2(n_in / n_out))) - 2
    quarter = n_in // 4
    parts = [_offline_express(K, V, vmax, x[:quarter], n_out, mbar, delta, seed, head)]
    dm = 0.5 * delta * (1 / math.log2(m / 2 + 2) - 1 / math.log2(m / 2 + 3))
    q = min(m, mbar)
    for j in (1, 2, 3):
        blk = list(x[j * quarter:(j + 1) * quarter])
        if m > mbar:                                   # Offline-Subsample: one uniform point per stratum
            w = 2 ** (m - mbar)
            code = 61 + 64 * (4 * (m // 2) + j)
            blk = [blk[s * w + int(math.floor(oracle.uniform(seed, s, 0, code, head) * w))] for s in range(len(blk) // w)]
        cur = blk
        for i in range(q):                             # Offline-Compress2(q, ., Halve_m)
            groups = 4 ** (q - 1 - i)
            gs = len(cur) // groups
            dlt = 4.0 ** (i + 1 - q) * dm / (3 * q)
            nxt = []
            for g in range(groups):
                xs = np.array(cur[g * gs:(g + 1) * gs], dtype=np.int32)
                U = np.array([oracle.uniform(seed, p, g, i + 64 * (4 * (m // 2) + j), head) for p in range(gs // 2)])
                nxt.extend(oracle.kh(K, V, vmax, xs, dlt, U)[0].tolist())
            cur = nxt
        parts.append(cur)
    E = np.array(sum(parts, []), dtype=np.int32)
    for h in (0, 1):
        U = np.array([oracle.uniform(seed, p, 0, 62 + h + 64 * (4 * (m // 2)), head) for p in range(len(E) // 2)])
        E = oracle.kh(K, V, vmax, E, 0.5 * dm, U)[0]
    return E.tolist()


@pytest.mark.parametrize("log2_nout,mbar,k", [(3, 2, 2), (2, 2, 3), (3, 1, 3)])
def test_streaming_equals_offline_express(log2_nout, mbar, k):
    n_out = 1 << log2_nout
    n = n_out * 4 ** k
    Q, K, V = _qkv(5, n, 4)
    r = oracle.thinformer_express(Q, K, V, log2_nout, mbar, seed=9, head=2, want_outputs=False)
    off = _offline_express(K, V, oracle.vmax(V), list(range(n)), n_out, mbar, 0.5, 9, 2)
    assert r["final_idx"].tolist() == off


def test_error_against_exact_causal_attention_is_moderate_and_seeded():
    Q, K, V = _qkv(6, 512, 8)
    a = oracle.thinformer_express(Q, K, V, 4, 2, seed=1)["O"]
    b = oracle.thinformer_express(Q, K, V, 4, 2, seed=1)["O"]
    c = oracle.thinformer_express(Q, K, V, 4, 2, seed=2)["O"]
    ex = oracle.exact_causal_attention(Q, K, V)
    assert np.array_equal(a, b) and not np.array_equal(a, c)
    # a larger cache approximates better (averaged over tokens)
    big = oracle.thinformer_express(Q, K, V, 6, 4, seed=1)["O"]
    assert np.abs(big - ex).mean() < np.abs(a - ex).mean()


# --------------------------------------------------------------------------------------
# Corollary 2's failure-probability schedule, read off the record of the oracle's own KH calls
# --------------------------------------------------------------------------------------
def _delta_m(delta, m):
    """Corollary 2: delta_m = (delta / 2) (1 / log2(m/2 + 2) - 1 / log2(m/2 + 3))."""
    return 0.5 * delta * (1.0 / math.log2(m / 2 + 2) - 1.0 / math.log2(m / 2 + 3))


@pytest.mark.parametrize("log2_nout,mbar,k,delta", [(3, 2, 3, 0.5), (2, 3, 4, 0.5), (3, 1, 3, 0.25), (2, 0, 3, 0.5),
                                                    (3, 4, 4, 0.9)])
def test_halve_calls_use_corollary_2_schedule(log2_nout, mbar, k, delta):
    """Every KH call the streaming oracle makes, with the delta it was given, against Corollary 2:
    Halve_{m,m} = KH(delta_m / 2) on 4 n_out and then 2 n_out points; Halve_{m,i} = KH(delta_{m,i}),
    delta_{m,i} = 4^(i+1-q) delta_m / (3 q), q = min(m, mbar), on n_out 2^(i+2-q) points (Algorithm 2's
    size rule with n_in = 2^q n_out), 4^(q-1-i) calls per sibling and three siblings per round."""
    n_out = 1 << log2_nout
    n = n_out * 4 ** k
    Q, K, V = _qkv(7, n, 3)
    log = oracle.thinformer_express(Q, K, V, log2_nout, mbar, delta=delta, want_outputs=False)["halve_log"]
    rounds = sorted(set(log[:, 0].astype(int).tolist()))
    assert rounds == [2 * r for r in range(k)]
    for m in rounds:
        rows = log[log[:, 0] == m]
        q = min(m, mbar)
        dm = _delta_m(delta, m)
        e_rows = rows[rows[:, 1] < 0]
        assert e_rows[:, 1].tolist() == [-1.0, -2.0]                       # twice, in this order, last in the round
        assert np.array_equal(rows[-2:], e_rows)
        assert e_rows[:, 2].tolist() == [4 * n_out, 2 * n_out]
        assert np.allclose(e_rows[:, 3], dm / 2, rtol=1e-13, atol=0)
        for j in (1, 2, 3):
            sib = rows[(rows[:, 1] >= 0) & (rows[:, 4] == j)]
            for i in range(q):
                lvl = sib[sib[:, 1] == i]
                assert len(lvl) == 4 ** (q - 1 - i)
                assert np.all(lvl[:, 2] == n_out * 2 ** (i + 2 - q))
                assert np.allclose(lvl[:, 3], 4.0 ** (i + 1 - q) * dm / (3 * q), rtol=1e-13, atol=0)
            assert len(sib) == sum(4 ** (q - 1 - i) for i in range(q))
        assert len(rows) == 2 + 3 * sum(4 ** (q - 1 - i) for i in range(q))


@pytest.mark.parametrize("log2_nout,mbar,k,delta", [(3, 2, 3, 0.5), (2, 3, 4, 0.5), (2, 1, 4, 0.7)])
def test_failure_budget_telescopes_as_in_corollary_2_proof(log2_nout, mbar, k, delta):
    """The proof of Corollary 2 charges KH(eta) a failure probability eta / 2 and shows that round m
    spends delta_m / 2 on the two halvings of E and (3/8) sum_i 4^(q-i) delta_{m,i} = delta_m / 2 on its
    three Compress2 instances, the rounds telescoping to
        sum_{even m <= M} delta_m = (delta / 2) (1 - 1 / log2(M/2 + 3))   (-> delta / 2).
    Summed here from the delta of every call the oracle made; a round with q = 0 makes no Compress2
    call and spends its first half only.  No formula of the schedule is retyped: a wrong logarithm
    base, a missing factor 1/2 in Halve_{m,m} or a shifted exponent in delta_{m,i} breaks the total."""
    n_out = 1 << log2_nout
    n = n_out * 4 ** k
    Q, K, V = _qkv(8, n, 3)
    log = oracle.thinformer_express(Q, K, V, log2_nout, mbar, delta=delta, want_outputs=False)["halve_log"]
    M = 2 * (k - 1)
    spent = 0.5 * log[:, 3].sum()
    closed = 0.5 * delta * (1.0 - 1.0 / math.log2(M / 2 + 3))
    first_half_only = 0.5 * sum(_delta_m(delta, m) for m in range(0, M + 1, 2) if min(m, mbar) == 0)
    assert spent == pytest.approx(closed - first_half_only, rel=1e-12)
    assert spent < delta / 2
    # per round: the two halves are equal (q >= 1)
    for m in range(2, M + 1, 2):
        rows = log[log[:, 0] == m]
        if min(m, mbar) >= 1:
            assert 0.5 * rows[rows[:, 1] < 0, 3].sum() == pytest.approx(0.5 * rows[rows[:, 1] >= 0, 3].sum(), rel=1e-12)
    # delta_0 = (delta/2)(1 - 1/log2 3): the first term of the telescoping sum, from the first round's calls
    assert log[0, 3] + log[1, 3] == pytest.approx(0.5 * delta * (1 - 1 / math.log2(3)), rel=1e-13)


# --------------------------------------------------------------------------------------
# Algorithm 5: the input token joins S_0 with S_0's weight
# --------------------------------------------------------------------------------------
@pytest.mark.parametrize("log2_nout,mbar,t", [(3, 2, 32 + 13), (3, 2, 32 + 32 + 5), (2, 1, 16 + 48 + 7), (2, 3, 64 + 64 + 21)])
def test_input_token_enters_with_weight_of_S0(log2_nout, mbar, t):
    """O[t] of the streaming run = the weighted softmax ratio over wtd_cache() as it stands when token t
    arrives, with (k_t, v_t) added to S_0, i.e. with S_0's weight 2^(-q) (Algorithm 5, "incorporate input
    token"; q = min(m, mbar) of the running Compress2).  The cache is taken from a second run of the oracle
    that stops after t updates; the ratio is recomputed here in NumPy.  With weight 1 instead (right only
    while q = 0) the outputs differ visibly."""
    n_out = 1 << log2_nout
    d = 4
    Q, K, V = _qkv(9, t + 9, d)
    V[0, 0] = 10.0                                  # v_max is reached in row 0: every prefix has the same kernel
    full = oracle.thinformer_express(Q, K, V, log2_nout, mbar, seed=3)
    pre = oracle.thinformer_express(Q[:t], K[:t], V[:t], log2_nout, mbar, seed=3, want_outputs=False)
    assert len(pre["final_idx"]) == full["cache_size"][t]
    m_t = 2 * math.ceil(math.log((t + 1) / (4 * n_out), 4) - 1e-12)     # thinning factor while token t+1 arrives
    q = min(m_t, mbar)
    assert q >= 1
    assert pre["final_w"].min() >= 2.0 ** -q
    idx = np.append(pre["final_idx"], t)
    K64, V64, q64 = K.astype(np.float64), V.astype(np.float64), Q[t].astype(np.float64)

    def ratio(w_self):
        w = np.append(pre["final_w"], w_self)
        e = w * np.exp(K64[idx] @ q64 / math.sqrt(d))
        return (e[:, None] * V64[idx]).sum(0) / e.sum()

    assert np.allclose(full["O"][t], ratio(2.0 ** -q), rtol=1e-11, atol=1e-13)
    assert np.abs(full["O"][t] - ratio(1.0)).max() > 1e-4
