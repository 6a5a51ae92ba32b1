"""elm_attend_static: the workspace-free variant of elm_attend for callers that must not
allocate device memory (the coreset operands are staged in an array built into the library).

Collected last on purpose.  Through the C ABI it checks the variant against the CPU oracle's
weighted attention at the bars of the attend parity tests, and against elm_attend bit for bit
(both run the same kernels), on calls in a row whose shapes differ: the shared array keeps the
previous call's bytes, so a later, smaller and ragged call shows that nothing stale is read.
It also checks that a warmed call leaves the device's free memory unchanged, that the status
word of the array reads 0, and that a request larger than the array is refused on the host.
"""
import ctypes

import numpy as np
import pytest
import torch

import paper_2606_10944_b200 as elm
from paper_2606_10944_b200 import binding
from paper_2606_10944_b200.workloads import WORKLOADS, generate

from _util import max_rel_err, oracle_attend

pytestmark = pytest.mark.gpu

TOL = {("f32", "fp64"): 2e-6, ("f32", "fp32"): 1e-4, ("bf16", "fp64"): 1e-2, ("bf16", "fp32"): 2e-2}


def _case(dtype, d, n, n_core, n_q, hq, hkv, seed):
    wl = WORKLOADS["cfg2"].scaled(batch=2, q_heads=hq, kv_heads=hkv, n=n, n_q=n_q, d=d, dtype=dtype)
    Qh, Kh, Vh = generate(wl, seed=seed)
    g = torch.Generator().manual_seed(seed)
    idx = torch.stack([torch.stack([torch.randperm(n, generator=g)[:n_core] for _ in range(hkv)])
                       for _ in range(2)]).to(torch.int32)
    w = torch.rand(2, hkv, n_core, generator=g) + 0.05
    return (Qh, Kh, Vh, idx, w), tuple(t.cuda() for t in (Qh, Kh, Vh, idx, w))


# (dtype, d, n, n_core, n_q, q heads, kv heads, seed), called in this order for each precision
CALLS = [
    ("f32", 128, 4096, 2000, 40, 4, 2, 1),      # fills 8 MiB of the array with fp32 rows
    ("bf16", 128, 4096, 300, 300, 8, 2, 2),     # tensor-core path, last block of 128 entries partly filled
    ("bf16", 128, 4096, 2048, 300, 8, 2, 3),    # tensor-core path, whole blocks
    ("f32", 64, 2048, 100, 77, 4, 2, 4),        # other head dimension, ragged
    ("bf16", 128, 4096, 700, 1, 8, 2, 5),       # one query and four query heads per KV head: the few-query kernels
]


def test_static_variant_matches_oracle_and_attend_on_consecutive_calls():
    for precision in ("fp32", "fp64"):
        for dtype, d, n, n_core, n_q, hq, hkv, seed in CALLS:
            host, dev = _case(dtype, d, n, n_core, n_q, hq, hkv, seed)
            Q, K, V, idx, w = dev
            out = torch.empty_like(Q)
            got = elm.attend_static(Q, K, V, idx, w, precision=precision, out=out)
            assert elm.attend_static_status(Q, K, n_core, precision) == 0
            ref = oracle_attend(host[0], host[1], host[2], host[3].numpy(), host[4].numpy().astype(np.float64))
            err = max_rel_err(got.float().cpu().numpy(), ref)
            assert err <= TOL[(dtype, precision)], (precision, dtype, n_core, err)
            same = elm.attend(Q, K, V, idx, w, precision=precision)
            torch.cuda.synchronize()
            assert torch.equal(got, same), (precision, dtype, n_core)


def test_static_variant_allocates_no_device_memory():
    _, (Q, K, V, idx, w) = _case("bf16", 128, 4096, 1024, 256, 8, 2, 6)
    out = torch.empty_like(Q)
    elm.attend_static(Q, K, V, idx, w, out=out)          # first call on the device: address look-up
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        elm.attend_static(Q, K, V, idx, w, out=out)
    assert elm.attend_static_status(Q, K, 1024) == 0
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before


def test_static_variant_refuses_oversized_coresets():
    lib = binding.load_library()
    _, (Q, K, V, idx, w) = _case("f32", 128, 16384, 8192, 8, 4, 4, 3)   # 2*4*8192*128*4 B * 2 = 64 MiB > 16 MiB
    O = torch.empty_like(Q)
    p, _ = binding.make_params(2, 4, 4, 16384, 8, 128, 14, 0, binding.ELM_F32, "fp32")
    rc = lib.elm_attend_static(Q.data_ptr(), K.data_ptr(), V.data_ptr(), idx.data_ptr(), w.data_ptr(),
                               8192, ctypes.byref(p), O.data_ptr(), None)
    assert rc == -9
    assert b"static scratch" in lib.elm_strerror(rc)
    st = ctypes.c_int32(0)
    assert lib.elm_attend_static_status(ctypes.byref(p), 8192, ctypes.byref(st), None) == -9
    with pytest.raises(binding.ElmError):
        elm.attend_static(Q, K, V, idx, w, out=O)
