"""Failure handling on the GPU, without hanging or faulting anything.

1. A bounded wait that runs out: one tensor-core elm_attend launch is told (through the test hook elm_debug_set)
   to expect arrivals on its "probabilities ready" barriers that nobody makes, with the time limit of the waits
   shortened to 20 ms.  The waits give up, the launch winds down, the status word reads non-zero; the next call on
   the same workspace is normal again and its status word reads 0.
2. A caller's row number outside [0, n_kv): the library built with -DELM_BOUNDS_CHECK reads row 0 instead and
   reports the fact through the status word; nothing traps.
"""
import ctypes

import numpy as np
import pytest
import torch

import paper_2606_10944_b200 as elm
from paper_2606_10944_b200 import binding, build
from paper_2606_10944_b200.workloads import WORKLOADS, generate

from _util import max_rel_err, oracle_attend

pytestmark = pytest.mark.gpu


def _case(seed=3, n=2048, n_core=512, n_q=700):
    wl = WORKLOADS["cfg5"].scaled(q_heads=4, kv_heads=2, n=n, n_q=n_q)
    Q, K, V = generate(wl, seed=seed)
    g = torch.Generator().manual_seed(seed)
    idx = torch.stack([torch.randperm(n, generator=g)[:n_core] for _ in range(2)]).reshape(1, 2, n_core).to(torch.int32)
    w = torch.rand(1, 2, n_core, generator=g) + 0.05
    return wl, (Q, K, V, idx, w)


def test_a_wait_that_runs_out_sets_the_status_word_and_the_next_call_is_clean():
    lib = binding.load_library()
    wl, host = _case()
    Q, K, V, idx, w = (t.cuda() for t in host)
    p, _ = elm.make_params(1, 4, 2, wl.n, wl.n_q, wl.d, wl.n.bit_length() - 1, 0, binding.ELM_BF16, "fp32")
    ws = torch.empty(elm.attend_workspace_bytes(p, idx.shape[-1]), dtype=torch.uint8, device="cuda")
    assert lib.elm_debug_set(0, 20_000_000) == 0                      # waits give up after 20 ms
    try:
        assert lib.elm_debug_set(1, 1) == 0                           # the next launch misses one arrival per barrier
        elm.attend(Q, K, V, idx, w, precision="fp32", workspace=ws)
        torch.cuda.synchronize()                                      # the launch ends by itself
        assert elm.attend_status(ws, p, idx.shape[-1]) != 0
    finally:
        assert lib.elm_debug_set(0, 2_000_000_000) == 0
    O = elm.attend(Q, K, V, idx, w, precision="fp32", workspace=ws)
    torch.cuda.synchronize()
    assert elm.attend_status(ws, p, idx.shape[-1]) == 0
    ref = oracle_attend(host[0], host[1], host[2], host[3].numpy(), host[4].numpy().astype(np.float64))
    assert max_rel_err(O.float().cpu().numpy(), ref) <= 2e-2
    assert lib.elm_debug_set(0, 10) != 0 and lib.elm_debug_set(7, 1) != 0     # limits and unknown hooks are refused


@pytest.mark.parametrize("dtype,precision", [("bf16", "fp32"), ("f32", "fp32")])
def test_bounds_check_build_reports_a_bad_row_number(dtype, precision):
    path = build.LIB_CHECK
    assert path.exists(), "libelm_check.so is built by paper_2606_10944_b200.build"
    chk = ctypes.CDLL(str(path))
    vp = ctypes.c_void_p
    chk.elm_attend.argtypes = [vp, vp, vp, vp, vp, ctypes.c_int32, ctypes.POINTER(binding.ElmParams), vp, vp,
                               ctypes.c_size_t, vp]
    chk.elm_attend_status.argtypes = [vp, ctypes.POINTER(binding.ElmParams), ctypes.c_int32,
                                      ctypes.POINTER(ctypes.c_int32), vp]
    chk.elm_attend_workspace_bytes.argtypes = [ctypes.POINTER(binding.ElmParams), ctypes.c_int32,
                                               ctypes.POINTER(ctypes.c_size_t)]
    wl, host = _case(seed=5, n=1024, n_core=200, n_q=300)
    if dtype == "f32":
        host = tuple(t.float() if t.dtype == torch.bfloat16 else t for t in host)
    Q, K, V, idx, w = (t.cuda() for t in host)
    code = binding.ELM_BF16 if dtype == "bf16" else binding.ELM_F32
    p, _ = elm.make_params(1, 4, 2, wl.n, wl.n_q, wl.d, 10, 0, code, precision)
    need = ctypes.c_size_t(0)
    assert chk.elm_attend_workspace_bytes(ctypes.byref(p), 200, ctypes.byref(need)) == 0
    ws = torch.empty(need.value, dtype=torch.uint8, device="cuda")
    O = torch.empty_like(Q)
    st = ctypes.c_int32(-1)

    def call(index):
        rc = chk.elm_attend(Q.data_ptr(), K.data_ptr(), V.data_ptr(), index.data_ptr(), w.data_ptr(), 200,
                            ctypes.byref(p), O.data_ptr(), ws.data_ptr(), ws.numel(), None)
        assert rc == 0
        torch.cuda.synchronize()
        assert chk.elm_attend_status(ws.data_ptr(), ctypes.byref(p), 200, ctypes.byref(st), None) == 0
        return st.value

    assert call(idx) == 0                                             # good row numbers: nothing to report
    ref = oracle_attend(host[0], host[1], host[2], host[3].numpy(), host[4].numpy().astype(np.float64))
    assert max_rel_err(O.float().cpu().numpy(), ref) <= (2e-2 if dtype == "bf16" else 1e-4)
    bad = idx.clone()
    bad[0, 1, 17] = wl.n + 5                                          # one row number past the end
    assert call(bad) == 64
    bad[0, 1, 17] = -3
    assert call(bad) == 64
    assert call(idx) == 0                                             # and the word is clean again afterwards
