"""Helpers for the GPU parity tests: run the library on a workload, run the oracle, compare."""
import numpy as np
import torch

from oracle import ssm_oracle as O
from paper_2501_00692_b200 import binding as B
from paper_2501_00692_b200 import synth

PARAM = O.PARAM_GRADS
TOL = {"f32": 1e-4, "bf16": 2e-2}   # relative error bars: fp32 I/O, bf16 I/O with fp32 accumulation


def theta_f64(theta):
    return {k: synth.to_f64(v) for k, v in theta.items()}


def errors(got, want, floor=0.0):
    """(relative L2 error, max-abs error relative to max-abs of the oracle).

    `floor` is a lower bound on the reference magnitude used in both ratios (per element for the max, times
    sqrt(size) for the L2 norm): it is only needed where the reference is identically zero because terms cancel."""
    got = np.asarray(got, dtype=np.float64); want = np.asarray(want, dtype=np.float64)
    d = got - want
    l2 = np.linalg.norm(d.ravel()) / max(np.linalg.norm(want.ravel()), floor * np.sqrt(max(want.size, 1)), 1e-300)
    mx = np.abs(d).max() / max(np.abs(want).max(), floor, 1e-300)
    return l2, mx


def assert_close(got, want, tol, what="", floor=0.0):
    assert np.isfinite(np.asarray(got, dtype=np.float64)).all(), f"{what}: non-finite values"
    l2, mx = errors(got, want, floor)
    assert l2 <= tol and mx <= tol, f"{what}: rel-L2 {l2:.3e}, rel-max {mx:.3e} > {tol}"
    return l2, mx


def gpu_adjoint(w, theta, x, dy, tbar, bptt=False, flags=0, grads=None, with_dx=True):
    dev = x.device
    sh = B.shape_of(x, w.d_state)
    _, gbytes = B.as_workspace_bytes(sh, tbar)
    ws = B.alloc_workspace(gbytes, dev)
    g = B.alloc_grads(sh, dev, with_dx) if grads is None else grads
    if bptt:
        B.as_full_bptt_grad(sh, theta, x, dy, g, ws, flags)
    else:
        B.as_adjoint_grad(sh, theta, x, dy, tbar, g, ws, flags)
    assert B.as_check_status(ws) == 0
    torch.cuda.synchronize()
    return g


def gpu_forward(w, theta, x):
    sh = B.shape_of(x, w.d_state)
    fbytes, _ = B.as_workspace_bytes(sh, w.seqlen)
    ws = B.alloc_workspace(fbytes, x.device)
    y = torch.empty_like(x)
    B.as_ssm_forward(sh, theta, x, y, ws)
    torch.cuda.synchronize()
    return y


def oracle_adjoint(theta, x, dy, tbar, tier="block", channel_block=None):
    th = theta_f64(theta)
    return O.batched(O.adjoint_grad, th, synth.to_f64(x), synth.to_f64(dy), tbar, tier=tier,
                     channel_block=channel_block)


def compare_grads(g, ref, tol, keys=PARAM + ("dx",), zero_floor=None):
    """`zero_floor` maps a gradient name to the magnitude its error is measured against when the oracle's value
    is identically zero (see `errors`)."""
    res = {}
    for k in keys:
        if g.get(k) is None:
            continue
        fl = (zero_floor or {}).get(k, 0.0) if not np.any(ref[k]) else 0.0
        res[k] = assert_close(synth.to_f64(g[k]), ref[k], tol, k, floor=fl)
    return res
