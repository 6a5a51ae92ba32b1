"""The C-ABI library without a GPU: it loads, exports what include/elm.h declares, sizes
workspaces and rejects bad arguments on the host before anything could be launched."""
import ctypes
import os
import re

import pytest

import oracle
from paper_2606_10944_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "elm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(elm_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound():
    lib = binding.load_library()
    names = _declared()
    assert "elm_compress" in names and "elm_attend" in names and len(names) >= 10
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(binding.EXPORTED_SYMBOLS) == names


def test_version_and_strerror():
    lib = binding.load_library()
    assert binding.version() >= 100
    assert lib.elm_strerror(0) == b"ok"
    assert b"workspace" in lib.elm_strerror(-5)


def test_default_delta_levels_match_schedule():
    for m in (1, 2, 5, 6):
        got = binding.default_delta_levels(m, 0.5)
        assert got == pytest.approx(list(oracle.default_delta_levels(m, 0.5)), rel=1e-15)
        assert sum(4 ** (m - 1 - i) * got[i] for i in range(m)) == pytest.approx(0.5 / 3)


def _params(**kw):
    base = dict(batch=1, q_heads=4, kv_heads=2, n_kv=1024, n_q=100, d=64, log2_nout=7, m=3,
                dtype_code=binding.ELM_F32)
    base.update(kw)
    return binding.make_params(**base)[0]


def test_workspace_sizes_scale_with_precision():
    c64, a = binding.workspace_bytes(_params(precision="fp64"))
    c32, a2 = binding.workspace_bytes(_params(precision="fp32"))
    # the pair Gram dominates: n_out^2 entries per problem
    assert c64 > 2 * 128 * 128 * 8 and c32 > 2 * 128 * 128 * 4 and c64 > c32
    assert a == a2 >= 2 * 2 * 128 * 64 * 4


@pytest.mark.parametrize("kw,code", [
    (dict(d=96), -2), (dict(n_kv=1000), -2), (dict(q_heads=3), -2), (dict(m=4, log2_nout=5), -2),
    (dict(log2_nout=1, m=9, n_kv=1024), -2), (dict(dtype_code=7), -3), (dict(delta=0.0), -6), (dict(delta=1.0), -6),
])
def test_bad_params_are_rejected_on_the_host(kw, code):
    lib = binding.load_library()
    p = _params(**kw)
    c = ctypes.c_size_t(0)
    assert lib.elm_workspace_bytes(ctypes.byref(p), ctypes.byref(c), None) == code
    # compute entry points validate before touching any pointer or the device
    assert lib.elm_compress(256, 256, ctypes.byref(p), 1, 256, 256, 256, 1 << 40, None) == code


def test_null_alignment_and_workspace_errors():
    lib = binding.load_library()
    p = _params()
    assert lib.elm_compress(None, 256, ctypes.byref(p), 1, 256, 256, 256, 1 << 40, None) == -1
    assert lib.elm_compress(264, 256, ctypes.byref(p), 1, 256, 256, 256, 1 << 40, None) == -4
    assert lib.elm_compress(256, 256, ctypes.byref(p), 1, 256, 256, 256, 16, None) == -5
    assert lib.elm_attend(256, 256, 256, 256, 256, 0, ctypes.byref(p), 256, 256, 1 << 40, None) == -2
    assert lib.elm_attend(256, 256, 256, 256, 256, 8, ctypes.byref(p), 256, 256, 16, None) == -5
    bad = binding.make_params(1, 4, 2, 1024, 100, 64, 7, 3, binding.ELM_F32, delta_level=[0.1, 0.2, 1.5])[0]
    assert lib.elm_workspace_bytes(ctypes.byref(bad), None, None) == -6


def test_compute_call_without_a_device_fails_loudly():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    K = torch.zeros(1, 1, 64, 64)
    with pytest.raises(binding.ElmError):
        binding.compress(K, K, 4, 2)


# ----------------------------------------------------------------------------------------------
# host logic of the ragged-length, Express and streaming entry points (no device needed)
# ----------------------------------------------------------------------------------------------
def _level_sizes(n_mid, n_out, m):
    sizes, a = [], n_mid
    for i in range(m):
        thresh = (n_out << (m + i)) >> (2 * (m - 1))
        calls = a // thresh
        sizes.append(a - calls * thresh)
        a = calls * (thresh // 2)
    return sizes + [a]


@pytest.mark.parametrize("n,log2_nout,m,n_sink,n_window", [
    (500, 4, 5, 0, 0), (500, 4, 5, 32, 32), (120, 3, 4, 5, 0), (63, 3, 3, 0, 9), (14, 3, 0, 4, 4), (9, 3, 3, 4, 5),
    (121673, 11, 6, 32, 32), (131072, 11, 6, 0, 0)])
def test_ragged_count_is_the_closed_form_of_algorithm_2(n, log2_nout, m, n_sink, n_window):
    """elm_compress_ragged_count = sinks + window + the points Algorithm 2 leaves in S_0..S_m after the middle
    rows: level i makes floor(a_i / t_i) calls, t_i = n_in 2^i / 4^(m-1)."""
    p = _params(n_kv=n, log2_nout=log2_nout, m=m, q_heads=2)
    count, ws = binding.compress_ragged_count(p, n_sink, n_window)
    assert count == n_sink + n_window + sum(_level_sizes(n - n_sink - n_window, 1 << log2_nout, m))
    assert ws > 0
    if n == 131072:
        assert count == 1 << log2_nout                      # the full length: elm_compress's coreset size


@pytest.mark.parametrize("kw,sink,window,code", [
    (dict(n_kv=50, log2_nout=3, m=2), 0, 0, -2),             # 50 middle rows > n_in = 32
    (dict(n_kv=50, log2_nout=3, m=3), 30, 30, -2),           # sinks + window exceed the sequence
    (dict(n_kv=50, log2_nout=1, m=6), 0, 0, -2),             # level-0 stretches below one pair
    (dict(n_kv=50, log2_nout=3, m=3), -1, 0, -2),
    (dict(n_kv=50, log2_nout=3, m=3, delta=1.5), 0, 0, -6),
])
def test_ragged_rejects_bad_sizes_on_the_host(kw, sink, window, code):
    lib = binding.load_library()
    p = _params(**kw)
    assert lib.elm_compress_ragged_count(ctypes.byref(p), sink, window, None, None) == code
    assert lib.elm_compress_ragged(256, 256, ctypes.byref(p), sink, window, 1, 256, 256, 256, 1 << 40, None) == code


def test_attend_takes_any_sequence_length():
    """The attention calls read K and V through the index list: n_kv need not be n_out 2^m."""
    p = _params(n_kv=1000, log2_nout=0, m=0)
    assert binding.attend_workspace_bytes(p, 300) > 0
    lib = binding.load_library()
    need = ctypes.c_size_t(0)
    assert lib.elm_attend_workspace_bytes(ctypes.byref(p), 1001, ctypes.byref(need)) == -2     # n_core > n_kv
    assert lib.elm_attend_workspace_bytes(ctypes.byref(_params(n_kv=1000, d=96)), 10, ctypes.byref(need)) == -2


def test_express_and_stream_argument_checks():
    lib = binding.load_library()
    need = ctypes.c_size_t(0)
    ok = _params(n_kv=16 * 64, n_q=16 * 64, log2_nout=4, m=0)
    assert lib.elm_express_workspace_bytes(ctypes.byref(ok), 2, ctypes.byref(need)) == 0 and need.value > 0
    small = need.value
    # the prefill also holds the round's level lists, the window lists with their lifetimes and log-denominators
    assert lib.elm_express_prefill_workspace_bytes(ctypes.byref(ok), 2, ctypes.byref(need)) == 0 and need.value > small
    # a length that is not n_out 4^R
    bad = _params(n_kv=16 * 8, n_q=16 * 8, log2_nout=4, m=0)
    assert lib.elm_express_workspace_bytes(ctypes.byref(bad), 2, ctypes.byref(need)) == -2
    # level-0 Halve calls of a single point: Compress2 of depth 6 on 2^7 points
    deep = _params(n_kv=2 * 4 ** 4, n_q=2 * 4 ** 4, log2_nout=1, m=0)
    assert lib.elm_express_prefill_workspace_bytes(ctypes.byref(deep), 6, ctypes.byref(need)) == -2
    # one query per token in the prefill; one query per step in the stream
    assert lib.elm_express_prefill_workspace_bytes(ctypes.byref(_params(n_kv=1024, n_q=100, log2_nout=4, m=0)), 2,
                                                   ctypes.byref(need)) == -2
    assert lib.elm_stream_workspace_bytes(ctypes.byref(_params(n_kv=1024, n_q=2, log2_nout=4, m=0)), 2,
                                          ctypes.byref(need)) == -2
    assert lib.elm_stream_workspace_bytes(ctypes.byref(_params(n_kv=1024, n_q=1, log2_nout=4, m=0)), 2,
                                          ctypes.byref(need)) == 0 and need.value > 0
