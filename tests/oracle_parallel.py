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


def _fwd_block(args):
    delta, xs, Bm, Cm, A = args
    return O.scan_forward(delta, xs, Bm, Cm, A)[0]


_POOL = None


def pool(workers=None):
    global _POOL
    if _POOL is None:
        n = workers or max(1, min(8, len(os.sched_getaffinity(0)) // 2))
        _POOL = mp.get_context("spawn").Pool(n)
    return _POOL


def host_memory_gb():
    """Memory this process may still use: the smaller of the host's available memory and the cgroup's headroom."""
    avail = 1e9
    try:
        for line in open("/proc/meminfo"):
            if line.startswith("MemAvailable:"):
                avail = int(line.split()[1]) / 2 ** 20
    except OSError:
        pass
    try:
        lim = open("/sys/fs/cgroup/memory.max").read().strip()
        if lim != "max":
            avail = min(avail, (int(lim) - int(open("/sys/fs/cgroup/memory.current").read())) / 2 ** 30)
    except (OSError, ValueError):
        pass
    return avail


def map_bounded(fn, jobs, gb_per_job):
    """pool().map in rounds small enough that the jobs running at once fit in half of the memory available."""
    p = pool()
    n = int(max(1, min(p._processes, 0.5 * host_memory_gb() // max(gb_per_job, 1e-3))))
    out = []
    for i in range(0, len(jobs), n):
        part = jobs[i:i + n]
        out += p.map(fn, part, chunksize=1) if len(part) > 1 else [fn(part[0])]
    return out


def _scan_gb(T, channels, states):
    """Rough peak of one _block job: about seven [T, channels, states] fp64 arrays."""
    return 7 * T * channels * states * 8 / 2 ** 30


def channel_scans(theta, x, g, tbar, tier="block", channel_block=32, channels=None, want=()):
    """Per-channel results of one sequence for `channels` (default: all): y, du, dx_dir, dA_log per channel, and the
    channel sums dB, dC over the channels given.  Returns a dict of arrays indexed like `channels`."""
    u, delta, Bm, Cm, A = O.nets(theta, x)
    sel = np.arange(x.shape[1]) if channels is None else np.asarray(channels)
    jobs = []
    for p0 in range(0, len(sel), channel_block):
        s = sel[p0:p0 + channel_block]
        jobs.append((delta[:, s], x[:, s], u[:, s], g[:, s], Bm, Cm, A[s], tbar, tier, tuple(want)))
    res = map_bounded(_block, jobs, _scan_gb(x.shape[0], channel_block, A.shape[1]))
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


def ssm_forward(theta, x, channel_block=64):
    """`oracle.ssm_oracle.ssm_forward` with the channel blocks of the scan on worker processes."""
    u, delta, Bm, Cm, A = O.nets(theta, x)
    jobs = [(delta[:, p0:p0 + channel_block], x[:, p0:p0 + channel_block], Bm, Cm, A[p0:p0 + channel_block])
            for p0 in range(0, x.shape[1], channel_block)]
    res = map_bounded(_fwd_block, jobs, _scan_gb(x.shape[0], channel_block, A.shape[1]) / 2)
    return np.concatenate(res, axis=1)


def stack_grad(thetas, y0, g, tbar, mode="chained", store=None, channel_block=64):
    """`oracle.ssm_oracle.stack_grad` (block tier) for one sequence with each layer's scans on worker processes: the
    same sequence of oracle calls (rmsnorm, layer forward, adjoint_grad, rmsnorm_vjp) and the `store` hook at the same
    places.  Returns ({"grads": per-layer dicts, "yK": top activation}, G_0 or None)."""
    keep = (lambda a: a) if store is None else store
    ys, yhats = [y0], []
    for th in thetas:
        yhats.append(keep(O.rmsnorm(ys[-1])))
        ys.append(keep(ys[-1] + keep(ssm_forward(th, yhats[-1], channel_block))))
    K = len(thetas)
    grads = [None] * K
    G = g
    for k in range(K - 1, -1, -1):
        grads[k] = adjoint_grad(thetas[k], yhats[k], G if mode == "chained" else g, tbar, tier="block",
                                channel_block=channel_block)
        if mode == "chained":
            G = keep(G + O.rmsnorm_vjp(ys[k], keep(grads[k]["dx"])))
    return {"grads": grads, "yK": ys[-1]}, (G if mode == "chained" else None)
