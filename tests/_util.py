"""Helpers shared by the tests (metrics and oracle marshalling); no product arithmetic."""
import numpy as np
import torch

import oracle
from paper_2606_10944_b200.workloads import as_f32_numpy


def oracle_compress(K, V, log2_nout, m, seed=1, delta=0.5, delta_level=None):
    """K, V: torch [B, H, n, d] -> (idx [B,H,n_out] int32, w float64, margins [B*H])."""
    B, H, n, d = K.shape
    Kf = as_f32_numpy(K).reshape(B * H, n, d)
    Vf = as_f32_numpy(V).reshape(B * H, n, d)
    idx, w, mg = oracle.compress2_batched(Kf, Vf, log2_nout, m, delta=delta, delta_level=delta_level, seed=seed)
    return idx.reshape(B, H, -1), w.reshape(B, H, -1), mg


def oracle_attend(Q, K, V, idx, w):
    return oracle.wtd_attention_batched(as_f32_numpy(Q), as_f32_numpy(K), as_f32_numpy(V),
                                        np.asarray(idx, dtype=np.int32), np.asarray(w, dtype=np.float64))


def oracle_exact(Q, K, V):
    return oracle.exact_attention_batched(as_f32_numpy(Q), as_f32_numpy(K), as_f32_numpy(V))


def max_rel_err(got, ref):
    """max_j ||got_j - ref_j||_inf / ||ref_j||_inf over all query rows j."""
    got = np.asarray(got, dtype=np.float64).reshape(-1, got.shape[-1])
    ref = np.asarray(ref, dtype=np.float64).reshape(-1, ref.shape[-1])
    num = np.abs(got - ref).max(axis=1)
    den = np.abs(ref).max(axis=1)
    return float((num / den).max())


def e_max(approx, exact):
    """max_j ||approx_j - exact_j||_inf (the quantity Theorem 3 bounds)."""
    return float(np.abs(np.asarray(approx, dtype=np.float64) - np.asarray(exact, dtype=np.float64)).max())


def e_fro(approx, exact):
    a = np.asarray(approx, dtype=np.float64)
    e = np.asarray(exact, dtype=np.float64)
    return float(np.linalg.norm(a - e) / np.linalg.norm(e))


def mismatch_rate(idx_a, idx_b):
    """1 - |A ∩ B| / n_out per problem, averaged."""
    a = np.asarray(idx_a).reshape(-1, idx_a.shape[-1])
    b = np.asarray(idx_b).reshape(-1, idx_b.shape[-1])
    return float(np.mean([1.0 - len(set(x.tolist()) & set(y.tolist())) / a.shape[1] for x, y in zip(a, b)]))


def check_coreset_structure(idx, n, m):
    """Facts true of any Compress2 output: distinct rows, and output slot t holds a survivor of
    the contiguous input block [t 2^m, (t+1) 2^m)."""
    idx = np.asarray(idx)
    n_out = idx.shape[-1]
    assert n_out << m == n
    flat = idx.reshape(-1, n_out)
    for row in flat:
        assert row.min() >= 0 and row.max() < n
        assert np.array_equal(row >> m, np.arange(n_out))
