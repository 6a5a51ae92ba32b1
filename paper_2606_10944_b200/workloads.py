"""Seeded synthetic inputs for the five benchmark workloads.

This module only draws random tensors; it holds none of the method's arithmetic and is
the one module that both the CUDA path's callers and the CPU oracle's callers may use.
Every tensor is produced on the host from ``numpy.random.Generator(PCG64(seed))`` so the
same bytes reach both sides.  ``N(0, x)`` in a workload's description is read with ``x``
as the variance unless it says "std".
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    batch: int
    q_heads: int
    kv_heads: int
    n: int            # keys/values per head
    n_q: int          # queries per head
    d: int
    dtype: str        # "f32", "bf16" or "e4m3": storage type of Q, K, V (and of O, which is bf16 for "e4m3")
    g: int            # oversampling: coreset size 2^g * 2^floor(log2(n)/2)
    recipe: str

    @property
    def log2_nout(self) -> int:
        return int(math.log2(self.n)) // 2 + self.g

    @property
    def m(self) -> int:
        return int(math.log2(self.n)) - self.log2_nout

    @property
    def n_out(self) -> int:
        return 1 << self.log2_nout

    def scaled(self, **kw) -> "Workload":
        """A smaller (or otherwise modified) instance of the same recipe."""
        return replace(self, **kw)


WORKLOADS = {
    "cfg1": Workload("cfg1", 1, 1, 1, 1024, 1024, 64, "f32", 0, "iid"),
    "cfg2": Workload("cfg2", 4, 12, 12, 1024, 1024, 64, "f32", 2, "mixture16"),
    "cfg3": Workload("cfg3", 2, 32, 32, 8192, 8192, 128, "bf16", 2, "lowrank8"),
    "cfg4": Workload("cfg4", 1, 32, 32, 32768, 32768, 128, "bf16", 3, "rope"),
    "cfg5": Workload("cfg5", 1, 32, 8, 131072, 131072, 128, "bf16", 3, "mixture64_t3"),
}


def _normal(rng, shape, std=1.0):
    x = rng.standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        x *= np.float32(std)
    return x


def _keys_values(rng, recipe: str, n: int, d: int):
    """K, V for one attention problem as float32 [n, d]."""
    if recipe == "iid":
        std = (1.0 / math.sqrt(d)) ** 0.5
        return _normal(rng, (n, d), std), _normal(rng, (n, d), std)
    if recipe == "mixture16":
        mu = _normal(rng, (16, d))
        comp = rng.integers(0, 16, size=n)
        K = mu[comp] + _normal(rng, (n, d), 0.3)
        return K, _normal(rng, (n, d))
    if recipe == "lowrank8":
        out = []
        for _ in range(2):
            W = _normal(rng, (8, d), math.sqrt(1.0 / 8.0))
            Z = _normal(rng, (n, 8))
            out.append(Z @ W + _normal(rng, (n, d), math.sqrt(0.1)))
        return out[0], out[1]
    if recipe == "rope":
        x = _normal(rng, (n, d)).astype(np.float64)
        pos = np.arange(n, dtype=np.float64)[:, None]
        t = np.arange(d // 2, dtype=np.float64)[None, :]
        ang = pos * (10000.0 ** (-2.0 * t / d))
        c, s = np.cos(ang), np.sin(ang)
        K = np.empty_like(x)
        K[:, 0::2] = x[:, 0::2] * c - x[:, 1::2] * s
        K[:, 1::2] = x[:, 0::2] * s + x[:, 1::2] * c
        return K.astype(np.float32), _normal(rng, (n, d))
    if recipe == "mixture64_t3":
        mu = _normal(rng, (64, d))
        comp = rng.integers(0, 64, size=n)
        K = mu[comp] + _normal(rng, (n, d), 0.3)
        t = rng.standard_t(3.0, size=n).astype(np.float32)
        K *= np.abs(t)[:, None]
        return K, _normal(rng, (n, d))
    raise ValueError(f"unknown recipe {recipe!r}")


def torch_dtype(name: str):
    return {"f32": torch.float32, "bf16": torch.bfloat16, "e4m3": torch.float8_e4m3fn}[name]


E4M3_MAX = 448.0      # largest finite E4M3 value: the draws are clamped to it before rounding (the format has no infinity)


def _store(x: torch.Tensor, dt):
    if dt == torch.float8_e4m3fn:
        return x.clamp_(-E4M3_MAX, E4M3_MAX).to(dt)
    return x.to(dt)


def generate(wl: Workload, seed: int = 1234, want_q: bool = True):
    """Return (Q, K, V) as CPU torch tensors in the workload's storage dtype.

    Shapes: Q [B, Hq, n_q, d]; K, V [B, Hkv, n, d].  Values are rounded to the storage
    dtype here, so both the CUDA path and the oracle (after an exact upcast) see the same
    numbers.  ``Q`` is ``None`` when ``want_q`` is false.
    """
    dt = torch_dtype(wl.dtype)
    # drawn in the order (K, V per problem) then Q per head, whatever the storage type; 16-bit and wider types are
    # rounded head by head, the 8-bit type (which torch cannot assign slice-wise) at the end
    mid = torch.float32 if dt == torch.float8_e4m3fn else dt
    rng = np.random.default_rng(np.random.PCG64(seed))
    K = torch.empty((wl.batch, wl.kv_heads, wl.n, wl.d), dtype=mid)
    V = torch.empty_like(K)
    for b in range(wl.batch):
        for h in range(wl.kv_heads):
            k, v = _keys_values(rng, wl.recipe, wl.n, wl.d)
            K[b, h] = torch.from_numpy(k).to(mid)
            V[b, h] = torch.from_numpy(v).to(mid)
    Q = None
    if want_q:
        qstd = (1.0 / math.sqrt(wl.d)) ** 0.5
        Q = torch.empty((wl.batch, wl.q_heads, wl.n_q, wl.d), dtype=mid)
        for b in range(wl.batch):
            for h in range(wl.q_heads):
                Q[b, h] = torch.from_numpy(_normal(rng, (wl.n_q, wl.d), qstd)).to(mid)
    if mid != dt:
        K, V = _store(K, dt), _store(V, dt)
        Q = _store(Q, dt) if Q is not None else None
    return Q, K, V


def as_f32_numpy(t: torch.Tensor) -> np.ndarray:
    """Exact upcast of an fp32 / bf16 / E4M3 tensor to a float32 NumPy array (for the oracle)."""
    return t.detach().to("cpu", torch.float32).contiguous().numpy()
