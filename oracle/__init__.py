"""CPU oracle (test infrastructure, never on the product path).

Thin ctypes wrapper around ``elm_oracle.c``: it converts NumPy arrays to pointers and
nothing else.  All arithmetic lives in the C file, in fp64, written from the paper
(Algorithm A.1, Offline-Compress2, Algorithm 5, Eq. katt, Eq. unmaskedatt).

Only ``tests/``, ``__graft_entry__.smoke()`` and the benchmark's CPU-baseline leg may
import this package.  It imports nothing from the CUDA package.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "elm_oracle.c"
_LIB = _HERE / "libelm_oracle.so"
_lib = None


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc (-O2, OpenMP over independent attention problems)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".tmp{os.getpid()}.so")
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-Wall", "-Wextra",
               "-o", str(tmp), str(_SRC), "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


_f32p = ctypes.POINTER(ctypes.c_float)
_f64p = ctypes.POINTER(ctypes.c_double)
_i32p = ctypes.POINTER(ctypes.c_int32)
_u32p = ctypes.POINTER(ctypes.c_uint32)


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(str(build()))
    lib.oracle_philox4x32_10.argtypes = [_u32p, _u32p, _u32p]
    lib.oracle_philox4x32_10.restype = None
    lib.oracle_uniform.argtypes = [ctypes.c_uint64] + [ctypes.c_uint32] * 4
    lib.oracle_uniform.restype = ctypes.c_double
    lib.oracle_vmax.argtypes = [_f32p, ctypes.c_int64, ctypes.c_int]
    lib.oracle_vmax.restype = ctypes.c_double
    lib.oracle_katt.argtypes = [_f32p, _f32p, ctypes.c_int, ctypes.c_double, ctypes.c_int64,
                                ctypes.c_int64, ctypes.c_double, ctypes.c_int]
    lib.oracle_katt.restype = ctypes.c_double
    lib.oracle_kh.argtypes = [_f32p, _f32p, ctypes.c_int, ctypes.c_double, _i32p, ctypes.c_int,
                              ctypes.c_double, ctypes.c_int, _f64p, _i32p, _i32p, _f64p]
    lib.oracle_kh.restype = ctypes.c_int
    lib.oracle_default_delta_levels.argtypes = [ctypes.c_int, ctypes.c_double, _f64p]
    lib.oracle_default_delta_levels.restype = None
    lib.oracle_compress2.argtypes = [_f32p, _f32p, ctypes.c_int64, ctypes.c_int, ctypes.c_int,
                                     ctypes.c_int, ctypes.c_double, _f64p, ctypes.c_uint64,
                                     ctypes.c_uint32, _i32p, _f64p, _f64p]
    lib.oracle_compress2.restype = ctypes.c_int
    lib.oracle_compress2_calls.argtypes = lib.oracle_compress2.argtypes + [_f64p, ctypes.c_int64,
                                                                           ctypes.POINTER(ctypes.c_int64)]
    lib.oracle_compress2_calls.restype = ctypes.c_int
    lib.oracle_compress2_batched.argtypes = [_f32p, _f32p, ctypes.c_int, ctypes.c_int64,
                                             ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                             ctypes.c_double, _f64p, ctypes.c_uint64, _i32p,
                                             _f64p, _f64p]
    lib.oracle_compress2_batched.restype = ctypes.c_int
    lib.oracle_compress2_stream.argtypes = [_f32p, _f32p, ctypes.c_int64, ctypes.c_int, ctypes.c_int,
                                            ctypes.c_int, ctypes.c_double, _f64p, ctypes.c_uint64,
                                            ctypes.c_uint32, ctypes.c_int32, ctypes.c_int32, _i32p, _f64p,
                                            ctypes.c_int32, _i32p]
    lib.oracle_compress2_stream.restype = ctypes.c_int
    lib.oracle_wtd_attention.argtypes = [_f32p, _f32p, _f32p, _i32p, _f64p, ctypes.c_int,
                                         ctypes.c_int64, ctypes.c_int, _f64p]
    lib.oracle_wtd_attention.restype = ctypes.c_int
    lib.oracle_exact_attention.argtypes = [_f32p, _f32p, _f32p, ctypes.c_int64, ctypes.c_int64,
                                           ctypes.c_int, _f64p]
    lib.oracle_exact_attention.restype = ctypes.c_int
    lib.oracle_wtd_attention_batched.argtypes = [_f32p, _f32p, _f32p, _i32p, _f64p, ctypes.c_int,
                                                 ctypes.c_int, ctypes.c_int, ctypes.c_int64,
                                                 ctypes.c_int64, ctypes.c_int, ctypes.c_int, _f64p]
    lib.oracle_wtd_attention_batched.restype = ctypes.c_int
    lib.oracle_exact_attention_batched.argtypes = [_f32p, _f32p, _f32p, ctypes.c_int, ctypes.c_int,
                                                   ctypes.c_int, ctypes.c_int64, ctypes.c_int64,
                                                   ctypes.c_int, _f64p]
    lib.oracle_exact_attention_batched.restype = ctypes.c_int
    lib.oracle_mmd2.argtypes = [_f32p, _f32p, ctypes.c_int, ctypes.c_double, _i32p, ctypes.c_int,
                                _i32p, _f64p, ctypes.c_int, ctypes.c_double]
    lib.oracle_mmd2.restype = ctypes.c_double
    _i64p = ctypes.POINTER(ctypes.c_int64)
    lib.oracle_thinformer_express.argtypes = [_f32p, _f32p, _f32p, ctypes.c_int64, ctypes.c_int, ctypes.c_int,
                                              ctypes.c_int, ctypes.c_double, ctypes.c_uint64, ctypes.c_uint32,
                                              _f64p, _i32p, _i32p, _f64p, _i32p, _i64p]
    lib.oracle_thinformer_express.restype = ctypes.c_int
    lib.oracle_thinformer_express_log.argtypes = lib.oracle_thinformer_express.argtypes + [_f64p, ctypes.c_int64]
    lib.oracle_thinformer_express_log.restype = ctypes.c_int
    lib.oracle_exact_causal_attention.argtypes = [_f32p, _f32p, _f32p, ctypes.c_int64, ctypes.c_int, _f64p]
    lib.oracle_exact_causal_attention.restype = ctypes.c_int
    lib.oracle_num_threads.argtypes = []
    lib.oracle_num_threads.restype = ctypes.c_int
    _lib = lib
    return lib


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a, a.ctypes.data_as(_f32p)


def _f64(a):
    a = np.ascontiguousarray(a, dtype=np.float64)
    return a, a.ctypes.data_as(_f64p)


def _i32(a):
    a = np.ascontiguousarray(a, dtype=np.int32)
    return a, a.ctypes.data_as(_i32p)


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def philox4x32_10(ctr, key):
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.uint32)
    _load().oracle_philox4x32_10(c.ctypes.data_as(_u32p), k.ctypes.data_as(_u32p),
                                 out.ctypes.data_as(_u32p))
    return out


def uniform(seed: int, pair: int, group: int, level: int, head: int) -> float:
    return float(_load().oracle_uniform(seed, pair, group, level, head))


def vmax(V) -> float:
    V, vp = _f32(V)
    return float(_load().oracle_vmax(vp, V.shape[0], V.shape[1]))


def katt(K, V, vmax_: float, a: int, b: int, shift: float = 0.0, use_floor: bool = False) -> float:
    K, kp = _f32(K)
    V, vp = _f32(V)
    return float(_load().oracle_katt(kp, vp, K.shape[1], vmax_, a, b, shift, int(use_floor)))


def kh(K, V, vmax_: float, x, delta: float, U, shift_mode: int = 1):
    """Algorithm A.1 on the point sequence ``x``; returns (S1, S2, diag[s/2, 4])."""
    K, kp = _f32(K)
    V, vp = _f32(V)
    x, xp = _i32(x)
    U, up = _f64(U)
    s = x.shape[0]
    assert U.shape[0] == s // 2
    S1 = np.zeros(s // 2, dtype=np.int32)
    S2 = np.zeros(s // 2, dtype=np.int32)
    diag = np.zeros((s // 2, 4), dtype=np.float64)
    rc = _load().oracle_kh(kp, vp, K.shape[1], vmax_, xp, s, delta, shift_mode, up,
                           S1.ctypes.data_as(_i32p), S2.ctypes.data_as(_i32p),
                           diag.ctypes.data_as(_f64p))
    if rc != 0:
        raise ValueError(f"oracle_kh failed with {rc}")
    return S1, S2, diag


def default_delta_levels(m: int, delta: float):
    out = np.zeros(max(m, 1), dtype=np.float64)
    _load().oracle_default_delta_levels(m, delta, out.ctypes.data_as(_f64p))
    return out[:m]


def compress2(K, V, log2_nout: int, m: int, delta: float = 0.5, delta_level=None, seed: int = 1,
              head: int = 0):
    """Offline-Compress2 on one attention problem; K, V are [n, d].

    Returns (idx[n_out] int32, w[n_out] float64, min_margin)."""
    K, kp = _f32(K)
    V, vp = _f32(V)
    n, d = K.shape
    n_out = 1 << log2_nout
    idx = np.zeros(n_out, dtype=np.int32)
    w = np.zeros(n_out, dtype=np.float64)
    mg = ctypes.c_double(0.0)
    dl = None
    if delta_level is not None:
        dl_arr, dl = _f64(delta_level)
        assert dl_arr.shape[0] == m
    rc = _load().oracle_compress2(kp, vp, n, d, log2_nout, m, delta, dl, seed, head,
                                  idx.ctypes.data_as(_i32p), w.ctypes.data_as(_f64p),
                                  ctypes.byref(mg))
    if rc != 0:
        raise ValueError(f"oracle_compress2 failed with {rc}")
    return idx, w, float(mg.value)


def compress2_calls(K, V, log2_nout: int, m: int, delta: float = 0.5, delta_level=None, seed: int = 1,
                    head: int = 0):
    """Offline-Compress2 as ``compress2``, also returning the record of its Halve calls.

    Returns (idx, w, calls[n_calls, 4]): per call, in the order made, level, number of the call at
    its level, points in, delta used."""
    K, kp = _f32(K)
    V, vp = _f32(V)
    n, d = K.shape
    n_out = 1 << log2_nout
    idx = np.zeros(n_out, dtype=np.int32)
    w = np.zeros(n_out, dtype=np.float64)
    cap = sum(4 ** i for i in range(max(m, 1)))
    log = np.zeros((cap, 4), dtype=np.float64)
    cnt = ctypes.c_int64(0)
    dl = None
    if delta_level is not None:
        dl_arr, dl = _f64(delta_level)
        assert dl_arr.shape[0] == m
    rc = _load().oracle_compress2_calls(kp, vp, n, d, log2_nout, m, delta, dl, seed, head,
                                        idx.ctypes.data_as(_i32p), w.ctypes.data_as(_f64p), None,
                                        log.ctypes.data_as(_f64p), cap, ctypes.byref(cnt))
    if rc != 0:
        raise ValueError(f"oracle_compress2_calls failed with {rc}")
    assert cnt.value <= cap
    return idx, w, log[:cnt.value].copy()


def compress2_batched(K, V, log2_nout: int, m: int, delta: float = 0.5, delta_level=None,
                      seed: int = 1):
    """K, V are [problems, n, d] (problems = batch * kv_heads); head counter = problem index."""
    K, kp = _f32(K)
    V, vp = _f32(V)
    P, n, d = K.shape
    n_out = 1 << log2_nout
    idx = np.zeros((P, n_out), dtype=np.int32)
    w = np.zeros((P, n_out), dtype=np.float64)
    mg = np.zeros(P, dtype=np.float64)
    dl = None
    if delta_level is not None:
        dl_arr, dl = _f64(delta_level)
        assert dl_arr.shape[0] == m
    rc = _load().oracle_compress2_batched(kp, vp, P, n, d, log2_nout, m, delta, dl, seed,
                                          idx.ctypes.data_as(_i32p), w.ctypes.data_as(_f64p),
                                          mg.ctypes.data_as(_f64p))
    if rc != 0:
        raise ValueError(f"oracle_compress2_batched failed with {rc}")
    return idx, w, mg


def compress2_stream(K, V, log2_nout: int, m: int, n_sink: int = 0, n_window: int = 0, delta: float = 0.5,
                     delta_level=None, seed: int = 1, head: int = 0):
    """Algorithm 2 fed the middle rows one by one, sink / window rows kept; K, V are [n, d] with any n.

    Returns (idx[count] int32, w[count] float64): sinks, S_0 .. S_m, window; weights sum to 1."""
    K, kp = _f32(K)
    V, vp = _f32(V)
    n, d = K.shape
    cap = n_sink + n_window + 5 * (1 << log2_nout) + 8 if m > 0 else n
    idx = np.zeros(cap, dtype=np.int32)
    w = np.zeros(cap, dtype=np.float64)
    cnt = ctypes.c_int32(0)
    dl = None
    if delta_level is not None:
        dl_arr, dl = _f64(delta_level)
        assert dl_arr.shape[0] == m
    rc = _load().oracle_compress2_stream(kp, vp, n, d, log2_nout, m, delta, dl, seed, head, n_sink, n_window,
                                         idx.ctypes.data_as(_i32p), w.ctypes.data_as(_f64p), cap,
                                         ctypes.byref(cnt))
    if rc != 0:
        raise ValueError(f"oracle_compress2_stream failed with {rc}")
    c = int(cnt.value)
    return idx[:c].copy(), w[:c].copy()


def wtd_attention(Q, K, V, idx, w):
    """Q [nq, d]; K, V [n, d]; idx, w [n_core] -> O [nq, d] float64."""
    Q, qp = _f32(Q)
    K, kp = _f32(K)
    V, vp = _f32(V)
    idx, ip = _i32(idx)
    w, wp = _f64(w)
    O = np.zeros(Q.shape, dtype=np.float64)
    rc = _load().oracle_wtd_attention(qp, kp, vp, ip, wp, idx.shape[0], Q.shape[0], Q.shape[1],
                                      O.ctypes.data_as(_f64p))
    if rc != 0:
        raise ValueError(f"oracle_wtd_attention failed with {rc}")
    return O


def exact_attention(Q, K, V):
    Q, qp = _f32(Q)
    K, kp = _f32(K)
    V, vp = _f32(V)
    O = np.zeros(Q.shape, dtype=np.float64)
    rc = _load().oracle_exact_attention(qp, kp, vp, K.shape[0], Q.shape[0], Q.shape[1],
                                        O.ctypes.data_as(_f64p))
    if rc != 0:
        raise ValueError(f"oracle_exact_attention failed with {rc}")
    return O


def wtd_attention_batched(Q, K, V, idx, w):
    """Q [B, Hq, nq, d]; K, V [B, Hkv, n, d]; idx, w [B, Hkv, n_core] -> O [B, Hq, nq, d]."""
    Q, qp = _f32(Q)
    K, kp = _f32(K)
    V, vp = _f32(V)
    idx, ip = _i32(idx)
    w, wp = _f64(w)
    B, Hq, nq, d = Q.shape
    Hkv, n = K.shape[1], K.shape[2]
    O = np.zeros(Q.shape, dtype=np.float64)
    rc = _load().oracle_wtd_attention_batched(qp, kp, vp, ip, wp, B, Hq, Hkv, n, nq, d,
                                              idx.shape[-1], O.ctypes.data_as(_f64p))
    if rc != 0:
        raise ValueError(f"oracle_wtd_attention_batched failed with {rc}")
    return O


def exact_attention_batched(Q, K, V):
    Q, qp = _f32(Q)
    K, kp = _f32(K)
    V, vp = _f32(V)
    B, Hq, nq, d = Q.shape
    Hkv, n = K.shape[1], K.shape[2]
    O = np.zeros(Q.shape, dtype=np.float64)
    rc = _load().oracle_exact_attention_batched(qp, kp, vp, B, Hq, Hkv, n, nq, d,
                                                O.ctypes.data_as(_f64p))
    if rc != 0:
        raise ValueError(f"oracle_exact_attention_batched failed with {rc}")
    return O


def mmd2(K, V, vmax_: float, in_idx, out_idx, w, shift: float = 0.0) -> float:
    K, kp = _f32(K)
    V, vp = _f32(V)
    a, ap = _i32(in_idx)
    o, op = _i32(out_idx)
    w, wp = _f64(w)
    return float(_load().oracle_mmd2(kp, vp, K.shape[1], vmax_, ap, a.shape[0], op, wp,
                                     o.shape[0], shift))


def thinformer_express(Q, K, V, log2_nout: int, mbar: int, delta: float = 0.5, seed: int = 1, head: int = 0,
                       want_outputs: bool = True):
    """Algorithms 1-5 streaming over one attention problem (Q, K, V are [n, d]).

    Returns a dict: O [n, d] (or None), cache_size [n] (points in wtd_cache() when token t arrives),
    final_idx / final_w (wtd_cache() after the last update), halve_calls, halve_log [halve_calls, 5]
    (per KH call in the order made: thinning factor m, level i or -1 / -2 for the two halvings of E,
    points in, delta used, sibling 1..3 or 0 for E)."""
    Q, qp = _f32(Q)
    K, kp = _f32(K)
    V, vp = _f32(V)
    n, d = K.shape
    n_out = 1 << log2_nout
    O = np.zeros((n, d), dtype=np.float64) if want_outputs else None
    cache = np.zeros(n, dtype=np.int32)
    fidx = np.zeros(6 * n_out + 1, dtype=np.int32)
    fw = np.zeros(6 * n_out + 1, dtype=np.float64)
    fc = ctypes.c_int32(0)
    hc = ctypes.c_int64(0)
    # a KH call consumes at least two points of its level and levels shrink by half: fewer than n calls
    log_cap = n + 8
    hlog = np.zeros((log_cap, 5), dtype=np.float64)
    rc = _load().oracle_thinformer_express_log(qp, kp, vp, n, d, log2_nout, mbar, delta, seed, head,
                                               O.ctypes.data_as(_f64p) if want_outputs else None,
                                               cache.ctypes.data_as(_i32p), fidx.ctypes.data_as(_i32p),
                                               fw.ctypes.data_as(_f64p), ctypes.byref(fc), ctypes.byref(hc),
                                               hlog.ctypes.data_as(_f64p), log_cap)
    if rc != 0:
        raise ValueError(f"oracle_thinformer_express failed with {rc}")
    c = int(fc.value)
    assert hc.value <= log_cap
    return {"O": O, "cache_size": cache, "final_idx": fidx[:c].copy(), "final_w": fw[:c].copy(),
            "halve_calls": int(hc.value), "halve_log": hlog[:int(hc.value)].copy()}


def exact_causal_attention(Q, K, V):
    Q, qp = _f32(Q)
    K, kp = _f32(K)
    V, vp = _f32(V)
    O = np.zeros(Q.shape, dtype=np.float64)
    rc = _load().oracle_exact_causal_attention(qp, kp, vp, K.shape[0], K.shape[1], O.ctypes.data_as(_f64p))
    if rc != 0:
        raise ValueError(f"oracle_exact_causal_attention failed with {rc}")
    return O
