"""Seeded synthetic inputs for the selective-SSM layer workloads.

This module only produces numbers: a counter-based generator (a 64-bit mixing
hash of (seed, element index) -> two uniforms -> Box-Muller) written in torch
integer/float64 ops so that it runs on the CPU or on a CUDA device, plus the
table of workload shapes.  It holds none of the method's arithmetic and is the
one module that both the CUDA binding's callers and the CPU oracle's callers
import.  Whoever generates a tensor is the source of truth for its bits: the
other side reads those bits (after the rounding to the I/O dtype done here),
it never regenerates them with a different math library.

Distributions (all workloads): x ~ N(0,1); dL/dy ~ N(0,1); W_B, W_C, W_delta ~
N(0, 1/d_model); b_delta ~ U(-4,-2) (``slow_decay``: U(-9,-7), which makes the
state decay slowly enough that a truncation window of thousands of tokens
changes the gradient visibly); A_log ~ U(0, ln 16) with A = -exp(A_log).
Seeds: ``1000*config + 17*layer + tensor_id``.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import torch

# tensor ids entering the seed
TID_X, TID_DY, TID_W_DELTA, TID_B_DELTA, TID_W_B, TID_W_C, TID_A_LOG = 1, 2, 3, 4, 5, 6, 7

_M1 = 0xBF58476D1CE4E5B9 - (1 << 64)  # as signed int64
_M2 = 0x94D049BB133111EB - (1 << 64)
_GOLD = 0x9E3779B97F4A7C15 - (1 << 64)


def _lsr(z: torch.Tensor, k: int) -> torch.Tensor:
    """Logical right shift of an int64 tensor."""
    return (z >> k) & ((1 << (64 - k)) - 1)


def _mix64(z: torch.Tensor) -> torch.Tensor:
    z = (z ^ _lsr(z, 30)) * _M1
    z = (z ^ _lsr(z, 27)) * _M2
    return z ^ _lsr(z, 31)


def _seed_offset(seed: int) -> int:
    """(seed + 1) * GOLD, wrapped to a signed 64-bit Python int."""
    v = ((int(seed) + 1) * _GOLD) & ((1 << 64) - 1)
    return v - (1 << 64) if v >= (1 << 63) else v


def uniform01(seed: int, start: int, count: int, device, stream_id: int = 0) -> torch.Tensor:
    """float64 uniforms in (0,1) for element indices [start, start+count)."""
    idx = torch.arange(start, start + count, dtype=torch.int64, device=device)
    z = _mix64(idx * 2 + stream_id + _seed_offset(seed))
    z = _mix64(z + _GOLD)
    k = _lsr(z, 11)  # 53 random bits
    return (k.to(torch.float64) + 0.5) * (1.0 / (1 << 53))


def normal(seed: int, start: int, count: int, device) -> torch.Tensor:
    """float64 standard normals (Box-Muller on two hashed uniforms per element)."""
    u1 = uniform01(seed, start, count, device, 0)
    u2 = uniform01(seed, start, count, device, 1)
    return torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)


def _fill(kind: str, seed: int, shape, device, dtype, scale=1.0, lo=0.0, hi=1.0,
          chunk: int = 1 << 26) -> torch.Tensor:
    n = 1
    for s in shape:
        n *= int(s)
    out = torch.empty(n, dtype=dtype, device=device)
    for start in range(0, n, chunk):
        cnt = min(chunk, n - start)
        if kind == "normal":
            v = normal(seed, start, cnt, device) * scale
        else:
            v = lo + (hi - lo) * uniform01(seed, start, cnt, device, 0)
        out[start:start + cnt] = v.to(dtype)
    return out.view(*shape)


@dataclass(frozen=True)
class Workload:
    """One synthetic workload: shapes, window, I/O dtype and seed base."""
    name: str
    config: int          # 1..5, enters the seed
    batch: int
    seqlen: int
    d_model: int
    d_state: int
    layers: int
    tbar: int            # >= seqlen means the full (untruncated) adjoint
    io: str              # "f32" or "bf16"

    @property
    def torch_dtype(self):
        return torch.float32 if self.io == "f32" else torch.bfloat16


# The five workloads (single layer unless `layers` > 1).
WORKLOADS = {
    "C1": Workload("C1", 1, 1, 512, 64, 16, 1, 512, "f32"),
    "C2": Workload("C2", 2, 1, 8192, 256, 16, 1, 64, "f32"),
    "C3": Workload("C3", 3, 2, 65536, 768, 16, 1, 2048, "bf16"),
    "C4": Workload("C4", 4, 2, 32768, 768, 16, 24, 1024, "bf16"),
    "C5": Workload("C5", 5, 1, 1048576, 2048, 16, 1, 4096, "bf16"),
}


def custom_workload(name, config, batch, seqlen, d_model, d_state=16, layers=1, tbar=None, io="f32"):
    return Workload(name, config, batch, seqlen, d_model, d_state, layers,
                    seqlen if tbar is None else tbar, io)


def layer_params(w: Workload, layer: int = 0, device="cpu", slow_decay: bool = False, b_delta_range=None) -> dict:
    """Parameters of layer `layer`: W_* in the I/O dtype, b_delta and A_log in fp32.
    `b_delta_range` (lo, hi) overrides the law of b_delta, e.g. (-1, 1) for a fast-decay corner (abar << 1)."""
    base = 1000 * w.config + 17 * layer
    P, N = w.d_model, w.d_state
    dt = w.torch_dtype
    std = 1.0 / math.sqrt(P)
    lo, hi = (-9.0, -7.0) if slow_decay else (-4.0, -2.0)
    if b_delta_range is not None:
        lo, hi = float(b_delta_range[0]), float(b_delta_range[1])
    return {
        "W_delta": _fill("normal", base + TID_W_DELTA, (P, P), device, dt, scale=std),
        "b_delta": _fill("uniform", base + TID_B_DELTA, (P,), device, torch.float32, lo=lo, hi=hi),
        "W_B": _fill("normal", base + TID_W_B, (N, P), device, dt, scale=std),
        "W_C": _fill("normal", base + TID_W_C, (N, P), device, dt, scale=std),
        "A_log": _fill("uniform", base + TID_A_LOG, (P, N), device, torch.float32,
                       lo=0.0, hi=math.log(16.0)),
    }


def activations(w: Workload, device="cpu"):
    """(x, dy), both [batch, seqlen, d_model] in the I/O dtype."""
    base = 1000 * w.config
    shape = (w.batch, w.seqlen, w.d_model)
    x = _fill("normal", base + TID_X, shape, device, w.torch_dtype)
    dy = _fill("normal", base + TID_DY, shape, device, w.torch_dtype)
    return x, dy


def to_f64(t: torch.Tensor):
    """Exact widening of a (possibly bf16, possibly CUDA) tensor to a float64 numpy array."""
    return t.detach().to("cpu").to(torch.float64).numpy()
