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
