"""Test harness only: run the fp64 oracle's per-channel scans on several host processes.

Channels are independent in the scans (only dB_t and dC_t sum over them), which is what
`oracle.ssm_oracle.adjoint_grad(channel_block=...)` already uses to bound memory.  Here the same blocks go to
worker processes.  Every number is produced by the oracle's own functions (`nets`, `scan_forward`, `mu_block`
/ `mu_direct`, `token_cotangents`, `_assemble`), composed in the order `adjoint_grad` composes them;
`tests/test_oracle_pins.py` checks that the result equals `adjoint_grad` itself.  Workers are spawned (not
forked), import numpy and the oracle only, and never touch CUDA.
"""
from __future__ import annotations

import multiprocessing as mp
import os

import numpy as np

from oracle import ssm_oracle as O


def _block(args):
    """One channel block: forward scan, summed cotangent, per-token cotangents.  Optionally also the per-(p, n) sum
    sum_i |Delta_i A mu_i h_i| that bounds the rounding of abar_i h_{i-1} when it is formed as h_i - bbar_i."""
    delta, xs, u, g, Bm, Cm, A, tbar, tier, want = args
    y, H, abar = O.scan_forward(delta, xs, Bm, Cm, A)
    mu = (O.mu_direct if tier == "direct" else O.mu_block)(abar, g, Cm, tbar)
    tok = O.token_cotangents(mu, H, abar, g, delta, xs, u, Bm, A)
    out = {"y": y, "du": tok["du"], "dx_dir": tok["dx_dir"], "dB": tok["dB"], "dC": tok["dC"], "dA_log": tok["dA_log"]}
    if "absq" in want:
        out["absq"] = np.einsum("tpn,tp->pn", np.abs(mu * H[1:]), delta) * np.abs(A)
    return out


_POOL = None


def pool(workers=None):
    global _POOL
    if _POOL is None:
        n = workers or max(1, min(8, len(os.sched_getaffinity(0)) // 2))
        _POOL = mp.get_context("spawn").Pool(n)
    return _POOL


def channel_scans(theta, x, g, tbar, tier="block", channel_block=32, channels=None, want=()):
    """Per-channel results of one sequence for `channels` (default: all): y, du, dx_dir, dA_log per channel, and the
    channel sums dB, dC over the channels given.  Returns a dict of arrays indexed like `channels`."""
    u, delta, Bm, Cm, A = O.nets(theta, x)
    sel = np.arange(x.shape[1]) if channels is None else np.asarray(channels)
    jobs = []
    for p0 in range(0, len(sel), channel_block):
        s = sel[p0:p0 + channel_block]
        jobs.append((delta[:, s], x[:, s], u[:, s], g[:, s], Bm, Cm, A[s], tbar, tier, tuple(want)))
    res = pool().map(_block, jobs) if len(jobs) > 1 else [_block(j) for j in jobs]
    out = {k: np.concatenate([r[k] for r in res], axis=1) for k in ("y", "du", "dx_dir")}
    out["dA_log"] = np.concatenate([r["dA_log"] for r in res], axis=0)
    out["dB"] = sum(r["dB"] for r in res)
    out["dC"] = sum(r["dC"] for r in res)
    if "absq" in want:
        out["absq"] = np.concatenate([r["absq"] for r in res], axis=0)
    return out


def adjoint_grad(theta, x, g, tbar, tier="block", channel_block=32, want=()):
    """`oracle.ssm_oracle.adjoint_grad` for one sequence with its channel blocks spread over worker processes."""
    if tbar < 1:
        raise ValueError("tbar must be >= 1")
    s = channel_scans(theta, x, g, tbar, tier, channel_block, want=want)
    out = O._assemble(theta, x, s["du"], s["dB"], s["dC"], s["dx_dir"], s["dA_log"])
    out["y"] = s["y"]
    if "absq" in want:
        out["absq"] = s["absq"]
    return out


def batched_adjoint_grad(theta, x, g, tbar, **kw):
    """x, g [B,T,P]: parameter gradients summed over the batch, per-token outputs stacked (as `oracle.batched`)."""
    outs = [adjoint_grad(theta, x[b], g[b], tbar, **kw) for b in range(x.shape[0])]
    res = {}
    for k in outs[0]:
        if k in O.PARAM_GRADS or k == "absq":
            res[k] = sum(o[k] for o in outs)
        else:
            res[k] = np.stack([o[k] for o in outs])
    return res
