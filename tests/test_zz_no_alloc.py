"""elm_attend_static: the workspace-free variant of elm_attend for callers that must not
allocate device memory (the coreset operands are staged in an array built into the library).

Collected last on purpose.  It checks, through the C ABI, that the variant reproduces
elm_attend on two calls in a row with different inputs (the shared array keeps the first
call's bytes, so the second call shows nothing stale is read), and that a request larger than
the built-in array is refused on the host with its own status code.
"""
import ctypes

import numpy as np
import pytest
import torch

import paper_2606_10944_b200 as elm
from paper_2606_10944_b200 import binding
from paper_2606_10944_b200.workloads import WORKLOADS, generate

from _util import max_rel_err

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-4, "bf16": 2e-2}     # the bars the attend parity tests use


def _case(dtype, d, n, n_core, n_q, hq, hkv, seed):
    wl = WORKLOADS["cfg2"].scaled(batch=2, q_heads=hq, kv_heads=hkv, n=n, n_q=n_q, d=d, dtype=dtype)
    Q, K, V = (t.cuda() for t in generate(wl, seed=seed))
    g = torch.Generator().manual_seed(seed)
    idx = torch.stack([torch.stack([torch.randperm(n, generator=g)[:n_core] for _ in range(hkv)])
                       for _ in range(2)]).to(torch.int32).cuda()
    w = (torch.rand(2, hkv, n_core, generator=g) + 0.05).cuda()
    return Q, K, V, idx, w


def test_static_variant_matches_attend_on_consecutive_calls():
    calls = [("bf16", 128, 4096, 2048, 300, 8, 2, 1),     # 4 MiB of gathered operands
             ("f32", 64, 2048, 100, 77, 4, 2, 2)]         # different dtype, smaller, ragged
    for precision in ("fp32", "fp64"):
        for dtype, d, n, n_core, n_q, hq, hkv, seed in calls:
            Q, K, V, idx, w = _case(dtype, d, n, n_core, n_q, hq, hkv, seed)
            ref = elm.attend(Q, K, V, idx, w, precision=precision)
            out = torch.empty_like(Q)
            got = elm.attend_static(Q, K, V, idx, w, precision=precision, out=out)
            torch.cuda.synchronize()
            err = max_rel_err(got.float().cpu().numpy(), ref.float().cpu().numpy())
            assert err <= TOL[dtype], (precision, dtype, err)


def test_static_variant_refuses_oversized_coresets():
    lib = binding.load_library()
    Q, K, V, idx, w = _case("f32", 128, 16384, 8192, 8, 4, 4, 3)   # 2*4*8192*128*4 B * 2 = 64 MiB > 16 MiB
    O = torch.empty_like(Q)
    p, _ = binding.make_params(2, 4, 4, 16384, 8, 128, 14, 0, binding.ELM_F32, "fp32")
    rc = lib.elm_attend_static(Q.data_ptr(), K.data_ptr(), V.data_ptr(), idx.data_ptr(), w.data_ptr(),
                               8192, ctypes.byref(p), O.data_ptr(), None)
    assert rc == -9
    assert b"static scratch" in lib.elm_strerror(rc)
    with pytest.raises(binding.ElmError):
        elm.attend_static(Q, K, V, idx, w, out=O)
