"""ctypes binding of the C-ABI CUDA library (argument marshalling only).

Each function mirrors one entry point declared in ``include/elm.h``.  PyTorch is used for
device memory and the current stream; every arithmetic step runs inside the library's
kernels.  There is no CPU fallback: if ``csrc/libelm.so`` has not been built, or no CUDA
device is present when a compute call is made, an :class:`ElmError` is raised.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import torch

ELM_F32, ELM_BF16, ELM_E4M3 = 0, 1, 2
PREC_FP64_DET, PREC_FP32 = 0, 1
_PRECISIONS = {"fp64": PREC_FP64_DET, "fp64_det": PREC_FP64_DET, "fp32": PREC_FP32,
               PREC_FP64_DET: PREC_FP64_DET, PREC_FP32: PREC_FP32}
STAGE_NAMES = ["prepass", "level_prep", "gram", "walk", "emit", "gather", "attend"]

EXPORTED_SYMBOLS = [
    "elm_workspace_bytes", "elm_default_delta_levels", "elm_compress", "elm_attend",
    "elm_attend_workspace_bytes", "elm_attend_static", "elm_attend_static_status", "elm_compress_ragged_count", "elm_compress_ragged", "elm_express_workspace_bytes", "elm_express_compress",
    "elm_express_prefill_workspace_bytes", "elm_express_prefill",
    "elm_stream_workspace_bytes", "elm_stream_init", "elm_stream_step", "elm_stream_steps", "elm_stream_cache",
    "elm_host_call_scratch_bytes", "elm_compress_attend_host",
    "elm_compress_status", "elm_attend_status", "elm_debug_set", "elm_debug_round_check", "elm_profile_enable", "elm_profile_read", "elm_launch_count", "elm_strerror", "elm_version",
]


class ElmError(RuntimeError):
    pass


class ElmParams(ctypes.Structure):
    _fields_ = [
        ("batch", ctypes.c_int32), ("q_heads", ctypes.c_int32), ("kv_heads", ctypes.c_int32),
        ("n_kv", ctypes.c_int32), ("n_q", ctypes.c_int32), ("d", ctypes.c_int32),
        ("log2_nout", ctypes.c_int32), ("m", ctypes.c_int32),
        ("dtype", ctypes.c_int32), ("precision", ctypes.c_int32),
        ("delta", ctypes.c_double), ("delta_level", ctypes.POINTER(ctypes.c_double)),
    ]


class ElmStream(ctypes.Structure):
    _fields_ = [
        ("n", ctypes.c_int64), ("ell", ctypes.c_int64), ("n_E", ctypes.c_int64),
        ("m", ctypes.c_int32), ("b", ctypes.c_int32), ("q", ctypes.c_int32), ("mbar", ctypes.c_int32),
        ("n_S", ctypes.c_int64 * 16), ("calls", ctypes.c_int64 * 16),
        ("n_known", ctypes.c_int64), ("seed", ctypes.c_uint64),
    ]


_lib = None


def library_path() -> Path:
    return Path(__file__).resolve().parent / "csrc" / "libelm.so"


def load_library():
    global _lib
    if _lib is not None:
        return _lib
    path = library_path()
    if not path.exists():
        raise ElmError(f"{path} is missing: build it with `python -m paper_2606_10944_b200.build` "
                       "(there is no CPU fallback)")
    lib = ctypes.CDLL(str(path))
    vp, sz = ctypes.c_void_p, ctypes.c_size_t
    pp = ctypes.POINTER(ElmParams)
    szp = ctypes.POINTER(sz)
    lib.elm_workspace_bytes.argtypes = [pp, szp, szp]
    lib.elm_default_delta_levels.argtypes = [ctypes.c_int32, ctypes.c_double, ctypes.POINTER(ctypes.c_double)]
    lib.elm_compress.argtypes = [vp, vp, pp, ctypes.c_uint64, vp, vp, vp, sz, vp]
    lib.elm_attend.argtypes = [vp, vp, vp, vp, vp, ctypes.c_int32, pp, vp, vp, sz, vp]
    lib.elm_attend_workspace_bytes.argtypes = [pp, ctypes.c_int32, szp]
    lib.elm_attend_static.argtypes = [vp, vp, vp, vp, vp, ctypes.c_int32, pp, vp, vp]
    lib.elm_attend_static_status.argtypes = [pp, ctypes.c_int32, ctypes.POINTER(ctypes.c_int32), vp]
    lib.elm_compress_ragged_count.argtypes = [pp, ctypes.c_int32, ctypes.c_int32, ctypes.POINTER(ctypes.c_int32), szp]
    lib.elm_compress_ragged.argtypes = [vp, vp, pp, ctypes.c_int32, ctypes.c_int32, ctypes.c_uint64, vp, vp, vp, sz, vp]
    lib.elm_express_workspace_bytes.argtypes = [pp, ctypes.c_int32, szp]
    lib.elm_express_compress.argtypes = [vp, vp, pp, ctypes.c_int32, ctypes.c_uint64, vp, vp, vp, sz, vp]
    lib.elm_express_prefill_workspace_bytes.argtypes = [pp, ctypes.c_int32, szp]
    lib.elm_express_prefill.argtypes = [vp, vp, vp, pp, ctypes.c_int32, ctypes.c_uint64, vp, vp, vp, vp, sz, vp]
    sp = ctypes.POINTER(ElmStream)
    lib.elm_stream_workspace_bytes.argtypes = [pp, ctypes.c_int32, szp]
    lib.elm_stream_init.argtypes = [sp, vp, vp, ctypes.c_int64, pp, ctypes.c_int32, ctypes.c_uint64, vp, sz, vp]
    lib.elm_stream_step.argtypes = [sp, vp, vp, vp, pp, vp, vp, sz, vp]
    lib.elm_stream_steps.argtypes = [sp, ctypes.c_int32, vp, vp, vp, pp, vp, vp, sz, vp]
    lib.elm_stream_cache.argtypes = [sp, pp, vp, vp, ctypes.POINTER(ctypes.c_int32), vp, sz, vp]
    lib.elm_host_call_scratch_bytes.argtypes = [pp, szp]
    lib.elm_compress_attend_host.argtypes = [vp, vp, vp, vp, vp, vp, pp, ctypes.c_uint64, vp, sz, vp]
    lib.elm_compress_status.argtypes = [vp, pp, ctypes.POINTER(ctypes.c_int32), vp]
    lib.elm_attend_status.argtypes = [vp, pp, ctypes.c_int32, ctypes.POINTER(ctypes.c_int32), vp]
    lib.elm_debug_set.argtypes = [ctypes.c_int32, ctypes.c_int64]
    lib.elm_debug_round_check.argtypes = [ctypes.POINTER(ElmParams), ctypes.c_int32, ctypes.c_int32, ctypes.c_uint64,
                                          ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_int64),
                                          ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_int64)]
    lib.elm_profile_enable.argtypes = [ctypes.c_int]
    lib.elm_profile_read.argtypes = [ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_int64), ctypes.c_int32]
    lib.elm_launch_count.argtypes = []
    lib.elm_launch_count.restype = ctypes.c_int64
    lib.elm_strerror.argtypes = [ctypes.c_int]
    lib.elm_strerror.restype = ctypes.c_char_p
    lib.elm_version.argtypes = []
    for name in EXPORTED_SYMBOLS:
        if name not in ("elm_launch_count", "elm_strerror"):
            getattr(lib, name).restype = ctypes.c_int
    _lib = lib
    return lib


def _check(rc: int, what: str):
    if rc != 0:
        raise ElmError(f"{what} failed: {load_library().elm_strerror(rc).decode()} ({rc})")


def _require_cuda(*tensors):
    if not torch.cuda.is_available():
        raise ElmError("no CUDA device: the library has no CPU fallback")
    for t in tensors:
        if not t.is_cuda or not t.is_contiguous():
            raise ElmError("tensors must be contiguous CUDA tensors")


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return ELM_F32
    if t.dtype == torch.bfloat16:
        return ELM_BF16
    if t.dtype == torch.float8_e4m3fn:
        return ELM_E4M3
    raise ElmError(f"unsupported dtype {t.dtype}")


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def make_params(batch, q_heads, kv_heads, n_kv, n_q, d, log2_nout, m, dtype_code, precision="fp32",
                delta=0.5, delta_level=None):
    """Fill an ``elm_params``; returns (params, keepalive) where keepalive owns delta_level."""
    p = ElmParams()
    p.batch, p.q_heads, p.kv_heads = batch, q_heads, kv_heads
    p.n_kv, p.n_q, p.d = n_kv, n_q, d
    p.log2_nout, p.m = log2_nout, m
    p.dtype, p.precision = dtype_code, _PRECISIONS[precision]
    p.delta = float(delta)
    keep = None
    if delta_level is not None:
        keep = (ctypes.c_double * len(delta_level))(*[float(x) for x in delta_level])
        p.delta_level = ctypes.cast(keep, ctypes.POINTER(ctypes.c_double))
    return p, keep


def version() -> int:
    return int(load_library().elm_version())


def default_delta_levels(m: int, delta: float = 0.5):
    out = (ctypes.c_double * max(m, 1))()
    _check(load_library().elm_default_delta_levels(m, delta, out), "elm_default_delta_levels")
    return [out[i] for i in range(m)]


def workspace_bytes(params: ElmParams):
    c, a = ctypes.c_size_t(0), ctypes.c_size_t(0)
    _check(load_library().elm_workspace_bytes(ctypes.byref(params), ctypes.byref(c), ctypes.byref(a)),
           "elm_workspace_bytes")
    return int(c.value), int(a.value)


def _workspace(nbytes: int, device):
    return torch.empty(max(nbytes, 256), dtype=torch.uint8, device=device)


def compress(K, V, log2_nout: int, m: int, seed: int = 1, precision="fp32", delta: float = 0.5,
             delta_level=None, workspace=None):
    """elm_compress: K, V [B, Hkv, n, d] -> (idx int32 [B, Hkv, n_out], w float32 [B, Hkv, n_out])."""
    lib = load_library()
    _require_cuda(K, V)
    B, H, n, d = K.shape
    p, keep = make_params(B, H, H, n, 1, d, log2_nout, m, _dtype_code(K), precision, delta, delta_level)
    need, _ = workspace_bytes(p)
    ws = workspace if workspace is not None else _workspace(need, K.device)
    n_out = 1 << log2_nout
    idx = torch.empty((B, H, n_out), dtype=torch.int32, device=K.device)
    w = torch.empty((B, H, n_out), dtype=torch.float32, device=K.device)
    _check(lib.elm_compress(K.data_ptr(), V.data_ptr(), ctypes.byref(p), seed, idx.data_ptr(),
                            w.data_ptr(), ws.data_ptr(), ws.numel(), _stream()), "elm_compress")
    return idx, w


def compress_ragged_count(params: ElmParams, n_sink: int = 0, n_window: int = 0):
    """elm_compress_ragged_count -> (entries per attention problem, workspace bytes)."""
    c, b = ctypes.c_int32(0), ctypes.c_size_t(0)
    _check(load_library().elm_compress_ragged_count(ctypes.byref(params), n_sink, n_window, ctypes.byref(c),
                                                    ctypes.byref(b)), "elm_compress_ragged_count")
    return int(c.value), int(b.value)


def compress_ragged(K, V, log2_nout: int, m: int, n_sink: int = 0, n_window: int = 0, seed: int = 1, precision="fp32",
                    delta: float = 0.5, delta_level=None, workspace=None):
    """elm_compress_ragged: K, V [B, Hkv, n, d] with any n -> (idx, w) [B, Hkv, count]: the sink rows,
    Compress2's weighted cache after the middle rows, the window rows."""
    lib = load_library()
    _require_cuda(K, V)
    B, H, n, d = K.shape
    p, keep = make_params(B, H, H, n, 1, d, log2_nout, m, _dtype_code(K), precision, delta, delta_level)
    count, need = compress_ragged_count(p, n_sink, n_window)
    ws = workspace if workspace is not None else _workspace(need, K.device)
    idx = torch.empty((B, H, max(count, 1)), dtype=torch.int32, device=K.device)[:, :, :count]
    w = torch.empty((B, H, max(count, 1)), dtype=torch.float32, device=K.device)[:, :, :count]
    _check(lib.elm_compress_ragged(K.data_ptr(), V.data_ptr(), ctypes.byref(p), n_sink, n_window, seed, idx.data_ptr(),
                                   w.data_ptr(), ws.data_ptr(), ws.numel(), _stream()), "elm_compress_ragged")
    return idx, w


def express_compress(K, V, log2_nout: int, mbar: int, seed: int = 1, precision="fp32", delta: float = 0.5,
                     workspace=None):
    """elm_express_compress: K, V [B, Hkv, n, d] with n = n_out 4^R -> (idx, w) of the Express cache
    after the whole sequence (Offline-Express with KH-Express failure parameters)."""
    lib = load_library()
    _require_cuda(K, V)
    B, H, n, d = K.shape
    p, _ = make_params(B, H, H, n, 1, d, log2_nout, 0, _dtype_code(K), precision, delta)
    need = ctypes.c_size_t(0)
    _check(lib.elm_express_workspace_bytes(ctypes.byref(p), mbar, ctypes.byref(need)), "elm_express_workspace_bytes")
    ws = workspace if workspace is not None else _workspace(int(need.value), K.device)
    n_out = 1 << log2_nout
    idx = torch.empty((B, H, n_out), dtype=torch.int32, device=K.device)
    w = torch.empty((B, H, n_out), dtype=torch.float32, device=K.device)
    _check(lib.elm_express_compress(K.data_ptr(), V.data_ptr(), ctypes.byref(p), mbar, seed, idx.data_ptr(),
                                    w.data_ptr(), ws.data_ptr(), ws.numel(), _stream()), "elm_express_compress")
    return idx, w


def express_prefill(Q, K, V, log2_nout: int, mbar: int, seed: int = 1, precision="fp32", delta: float = 0.5,
                    workspace=None, out=None):
    """elm_express_prefill: Q [B, Hq, n, d], K, V [B, Hkv, n, d] -> (O like Q, idx, w): every token attends
    over the Express cache as of its own position plus itself (Thinformer Express in prefill)."""
    lib = load_library()
    _require_cuda(Q, K, V)
    B, Hq, nq, d = Q.shape
    H, n = K.shape[1], K.shape[2]
    p, _ = make_params(B, Hq, H, n, nq, d, log2_nout, 0, _dtype_code(K), precision, delta)
    need = ctypes.c_size_t(0)
    _check(lib.elm_express_prefill_workspace_bytes(ctypes.byref(p), mbar, ctypes.byref(need)),
           "elm_express_prefill_workspace_bytes")
    ws = workspace if workspace is not None else _workspace(int(need.value), K.device)
    n_out = 1 << log2_nout
    O = out if out is not None else torch.empty_like(Q)
    idx = torch.empty((B, H, n_out), dtype=torch.int32, device=K.device)
    w = torch.empty((B, H, n_out), dtype=torch.float32, device=K.device)
    _check(lib.elm_express_prefill(Q.data_ptr(), K.data_ptr(), V.data_ptr(), ctypes.byref(p), mbar, seed, O.data_ptr(),
                                   idx.data_ptr(), w.data_ptr(), ws.data_ptr(), ws.numel(), _stream()),
           "elm_express_prefill")
    return O, idx, w


class Stream:
    """elm_stream_*: streaming Thinformer Express over K, V [B, Hkv, capacity, d] (one token per step)."""

    def __init__(self, K, V, q_heads: int, log2_nout: int, mbar: int, seed: int = 1, precision="fp32",
                 delta: float = 0.5, n_known=None):
        lib = load_library()
        _require_cuda(K, V)
        B, H, n, d = K.shape
        self.K, self.V = K, V
        self.params, _ = make_params(B, q_heads, H, n, 1, d, log2_nout, 0, _dtype_code(K), precision, delta)
        need = ctypes.c_size_t(0)
        _check(lib.elm_stream_workspace_bytes(ctypes.byref(self.params), mbar, ctypes.byref(need)),
               "elm_stream_workspace_bytes")
        self.ws = _workspace(int(need.value), K.device)
        self.state = ElmStream()
        _check(lib.elm_stream_init(ctypes.byref(self.state), K.data_ptr(), V.data_ptr(), n if n_known is None else n_known,
                                   ctypes.byref(self.params), mbar, seed, self.ws.data_ptr(), self.ws.numel(), _stream()),
               "elm_stream_init")

    def step(self, q_t, out=None):
        """q_t [B, Hq, 1, d] -> O_t; the token is row state.n of K and V."""
        O = out if out is not None else torch.empty_like(q_t)
        _check(load_library().elm_stream_step(ctypes.byref(self.state), q_t.data_ptr(), self.K.data_ptr(), self.V.data_ptr(),
                                              ctypes.byref(self.params), O.data_ptr(), self.ws.data_ptr(), self.ws.numel(),
                                              _stream()), "elm_stream_step")
        return O

    def steps(self, q_T, out=None):
        """q_T [T, B, Hq, 1, d] -> O_T of the same shape: T tokens by one library call (elm_stream_steps)."""
        O = out if out is not None else torch.empty_like(q_T)
        _check(load_library().elm_stream_steps(ctypes.byref(self.state), q_T.shape[0], q_T.data_ptr(), self.K.data_ptr(),
                                               self.V.data_ptr(), ctypes.byref(self.params), O.data_ptr(), self.ws.data_ptr(),
                                               self.ws.numel(), _stream()), "elm_stream_steps")
        return O

    def cache(self):
        """(idx int32 [B, Hkv, count], w float32 [B, Hkv, count]) of wtd_cache()."""
        p = self.params
        cap = 6 * (1 << p.log2_nout) + 1
        idx = torch.empty((p.batch, p.kv_heads, cap), dtype=torch.int32, device=self.K.device)
        w = torch.empty((p.batch, p.kv_heads, cap), dtype=torch.float32, device=self.K.device)
        count = ctypes.c_int32(0)
        # the library writes dense [problem][count] arrays at the front of the buffers
        _check(load_library().elm_stream_cache(ctypes.byref(self.state), ctypes.byref(p), idx.data_ptr(), w.data_ptr(),
                                               ctypes.byref(count), self.ws.data_ptr(), self.ws.numel(), _stream()),
               "elm_stream_cache")
        c = int(count.value)
        flat_i = idx.reshape(-1)[: p.batch * p.kv_heads * c].reshape(p.batch, p.kv_heads, c)
        flat_w = w.reshape(-1)[: p.batch * p.kv_heads * c].reshape(p.batch, p.kv_heads, c)
        return flat_i, flat_w


def attend_workspace_bytes(params: ElmParams, n_core: int) -> int:
    need = ctypes.c_size_t(0)
    _check(load_library().elm_attend_workspace_bytes(ctypes.byref(params), n_core, ctypes.byref(need)),
           "elm_attend_workspace_bytes")
    return int(need.value)


def attend(Q, K, V, idx, w, precision="fp32", workspace=None, out=None):
    """elm_attend: Q [B, Hq, nq, d]; K, V [B, Hkv, n, d]; idx, w [B, Hkv, n_core] -> O like Q."""
    lib = load_library()
    _require_cuda(Q, K, V, idx, w)
    B, Hq, nq, d = Q.shape
    Hkv, n = K.shape[1], K.shape[2]
    n_core = idx.shape[-1]
    if idx.dtype != torch.int32 or w.dtype != torch.float32:
        raise ElmError("idx must be int32 and w float32")
    # log2_nout / m only describe compression; any consistent pair passes validation
    p, _ = make_params(B, Hq, Hkv, n, nq, d, n.bit_length() - 1, 0, _dtype_code(Q), precision)
    need = ctypes.c_size_t(0)
    _check(lib.elm_attend_workspace_bytes(ctypes.byref(p), n_core, ctypes.byref(need)),
           "elm_attend_workspace_bytes")
    ws = workspace if workspace is not None else _workspace(int(need.value), Q.device)
    # 8-bit inputs: the output is bf16
    O = out if out is not None else torch.empty(Q.shape, dtype=torch.bfloat16 if Q.dtype == torch.float8_e4m3fn else Q.dtype,
                                                device=Q.device)
    _check(lib.elm_attend(Q.data_ptr(), K.data_ptr(), V.data_ptr(), idx.data_ptr(), w.data_ptr(),
                          n_core, ctypes.byref(p), O.data_ptr(), ws.data_ptr(), ws.numel(), _stream()),
           "elm_attend")
    return O


ATTEND_STATIC_SCRATCH_BYTES = 16 << 20


def attend_static(Q, K, V, idx, w, precision="fp32", out=None):
    """elm_attend_static: elm_attend without a workspace argument.

    For callers that may not allocate device memory: the coreset operands are staged in a
    fixed array inside the library (ATTEND_STATIC_SCRATCH_BYTES), so this wrapper allocates
    nothing when ``out`` is supplied.  Calls on one device share that array; do not let two of
    them overlap on the GPU.
    """
    lib = load_library()
    _require_cuda(Q, K, V, idx, w)
    B, Hq, nq, d = Q.shape
    Hkv, n = K.shape[1], K.shape[2]
    if idx.dtype != torch.int32 or w.dtype != torch.float32:
        raise ElmError("idx must be int32 and w float32")
    p, _ = make_params(B, Hq, Hkv, n, nq, d, n.bit_length() - 1, 0, _dtype_code(Q), precision)
    O = out if out is not None else torch.empty_like(Q)
    _check(lib.elm_attend_static(Q.data_ptr(), K.data_ptr(), V.data_ptr(), idx.data_ptr(), w.data_ptr(),
                                 idx.shape[-1], ctypes.byref(p), O.data_ptr(), _stream()),
           "elm_attend_static")
    return O


def attend_static_status(Q, K, n_core: int, precision="fp32") -> int:
    """elm_attend_static_status after an attend_static call with these tensors' shapes: 0 unless a bounded
    device wait expired during it."""
    B, Hq, nq, d = Q.shape
    Hkv, n = K.shape[1], K.shape[2]
    p, _ = make_params(B, Hq, Hkv, n, nq, d, n.bit_length() - 1, 0, _dtype_code(Q), precision)
    out = ctypes.c_int32(-1)
    _check(load_library().elm_attend_static_status(ctypes.byref(p), n_core, ctypes.byref(out), _stream()),
           "elm_attend_static_status")
    return int(out.value)


def compress_attend_host(Q, K, V, log2_nout: int, m: int, seed: int = 1, precision="fp32",
                         delta: float = 0.5, scratch=None, out=None, want_coreset=False):
    """elm_compress_attend_host: CPU tensors in, CPU tensor out; copies happen inside the call."""
    lib = load_library()
    if not torch.cuda.is_available():
        raise ElmError("no CUDA device: the library has no CPU fallback")
    for t in (Q, K, V):
        if t.is_cuda or not t.is_contiguous():
            raise ElmError("host call takes contiguous CPU tensors")
    B, Hq, nq, d = Q.shape
    Hkv, n = K.shape[1], K.shape[2]
    p, _ = make_params(B, Hq, Hkv, n, nq, d, log2_nout, m, _dtype_code(Q), precision, delta)
    need = ctypes.c_size_t(0)
    _check(lib.elm_host_call_scratch_bytes(ctypes.byref(p), ctypes.byref(need)), "elm_host_call_scratch_bytes")
    dev = torch.device("cuda", torch.cuda.current_device())
    sc = scratch if scratch is not None else _workspace(int(need.value), dev)
    O = out if out is not None else torch.empty_like(Q)
    n_out = 1 << log2_nout
    idx = torch.empty((B, Hkv, n_out), dtype=torch.int32) if want_coreset else None
    w = torch.empty((B, Hkv, n_out), dtype=torch.float32) if want_coreset else None
    _check(lib.elm_compress_attend_host(Q.data_ptr(), K.data_ptr(), V.data_ptr(), O.data_ptr(),
                                        idx.data_ptr() if want_coreset else None,
                                        w.data_ptr() if want_coreset else None,
                                        ctypes.byref(p), seed, sc.data_ptr(), sc.numel(), _stream()),
           "elm_compress_attend_host")
    return (O, idx, w) if want_coreset else O


def host_call_scratch_bytes(B, Hq, Hkv, n, nq, d, log2_nout, m, dtype, precision="fp32") -> int:
    code = ELM_BF16 if dtype == torch.bfloat16 else ELM_F32
    p, _ = make_params(B, Hq, Hkv, n, nq, d, log2_nout, m, code, precision)
    need = ctypes.c_size_t(0)
    _check(load_library().elm_host_call_scratch_bytes(ctypes.byref(p), ctypes.byref(need)),
           "elm_host_call_scratch_bytes")
    return int(need.value)


def compress_status(workspace, params: ElmParams) -> int:
    """elm_compress_status: 0 unless a bounded device wait expired during the last compress call."""
    out = ctypes.c_int32(-1)
    _check(load_library().elm_compress_status(workspace.data_ptr(), ctypes.byref(params), ctypes.byref(out), _stream()),
           "elm_compress_status")
    return int(out.value)


def attend_status(workspace, params: ElmParams, n_core: int) -> int:
    """elm_attend_status: 0 unless a bounded device wait expired during the last attend call."""
    out = ctypes.c_int32(-1)
    _check(load_library().elm_attend_status(workspace.data_ptr(), ctypes.byref(params), n_core, ctypes.byref(out),
                                            _stream()), "elm_attend_status")
    return int(out.value)


def debug_round_check(B, Hq, Hkv, n, d, log2_nout, mbar, r, seed=1, dtype_code=None, precision="fp32"):
    """elm_debug_round_check (host only): (missing, listed_blocks, needed_blocks, partly_blocks) for Express round r of a prefill, or
    None when that round does not take the one-launch form."""
    lib = load_library()
    p, _ = make_params(B, Hq, Hkv, n, n, d, log2_nout, 0, ELM_BF16 if dtype_code is None else dtype_code, precision)
    out = [ctypes.c_int64(0) for _ in range(4)]
    rc = lib.elm_debug_round_check(ctypes.byref(p), mbar, r, seed, *[ctypes.byref(o) for o in out])
    if rc == -2:                     # ELM_ERR_SHAPE: the round is taken in windows
        return None
    _check(rc, "elm_debug_round_check")
    return tuple(int(o.value) for o in out)


def profile_enable(on=True):
    """0 / False: off; 1 / True: every stage; 2: the attention stage only (see include/elm.h)."""
    _check(load_library().elm_profile_enable(int(on)), "elm_profile_enable")


def profile_read():
    """Per-stage (milliseconds, launches) since the last read, as a dict keyed by stage name."""
    n = len(STAGE_NAMES)
    ms = (ctypes.c_float * n)()
    ln = (ctypes.c_int64 * n)()
    _check(load_library().elm_profile_read(ms, ln, n), "elm_profile_read")
    return {STAGE_NAMES[i]: (float(ms[i]), int(ln[i])) for i in range(n)}


def launch_count() -> int:
    return int(load_library().elm_launch_count())
