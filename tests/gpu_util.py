"""Helpers for the GPU parity tests: run the library on a workload, run the oracle, compare."""
import numpy as np
import torch

from oracle import ssm_oracle as O
from paper_2501_00692_b200 import binding as B
from paper_2501_00692_b200 import synth

PARAM = O.PARAM_GRADS
TOL = {"f32": 1e-4, "bf16": 2e-2}   # relative error bars: fp32 I/O, bf16 I/O with fp32 accumulation


def bf16_round(a):
    """Round-to-nearest-even to bfloat16, returned as float64: the storage format of bf16 I/O."""
    return torch.from_numpy(np.ascontiguousarray(a)).to(torch.bfloat16).to(torch.float64).numpy()


def theta_f64(theta):
    return {k: synth.to_f64(v) for k, v in theta.items()}


def errors(got, want):
    """(relative L2 error, max-abs error relative to max-abs of the oracle)."""
    got = np.asarray(got, dtype=np.float64); want = np.asarray(want, dtype=np.float64)
    d = got - want
    l2 = np.linalg.norm(d.ravel()) / max(np.linalg.norm(want.ravel()), 1e-300)
    mx = np.abs(d).max() / max(np.abs(want).max(), 1e-300)
    return l2, mx


def assert_close(got, want, tol, what=""):
    assert np.isfinite(np.asarray(got, dtype=np.float64)).all(), f"{what}: non-finite values"
    l2, mx = errors(got, want)
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


def compare_grads(g, ref, tol, keys=PARAM + ("dx",)):
    res = {}
    for k in keys:
        if g.get(k) is None:
            continue
        res[k] = assert_close(synth.to_f64(g[k]), ref[k], tol, k)
    return res


EPS32 = 2.0 ** -24   # unit roundoff of fp32
DALOG_C = 4.0        # rounding units of h_i allowed per term (see assert_dalog_rows)


def oracle_adjoint_with_bound(theta, x, dy, tbar, tier="direct", channel_block=32, scalar_states=None):
    """Oracle gradients plus `absq`[p,n] = sum over tokens and batch of |Delta_i A mu_i h_i| (from the oracle's own
    mu and h): the scale of the rounding error of dA_log when abar_i h_{i-1} is formed from h_i.
    `scalar_states` = N selects the scalar structure (theta["A_log"] is [P]): the diagonal layer with tied rates."""
    import oracle_parallel as OP
    th = theta_f64(theta)
    if scalar_states:
        th = O.untie_scalar_A(th, scalar_states)
    ref = OP.batched_adjoint_grad(th, synth.to_f64(x), synth.to_f64(dy), tbar, tier=tier,
                                  channel_block=channel_block, want=("absq",))
    if scalar_states:
        ref["dA_log"] = ref["dA_log"].sum(axis=1)
    return ref


def compare_all(g, ref, tol):
    """Every gradient against the oracle; dA_log row by row with the rounding bound, and as a whole tensor too
    unless the oracle's dA_log is identically zero (a single token: h_0 = 0)."""
    keys = PARAM + ("dx",)
    if not np.any(ref["dA_log"]):
        keys = tuple(k for k in keys if k != "dA_log")
    compare_grads(g, ref, tol, keys)
    return assert_dalog_rows(synth.to_f64(g["dA_log"]), ref, tol)


def assert_dalog_rows(got, ref, tol, what="dA_log"):
    """dA_log channel by channel.  The library forms abar_i h_{i-1} as h_i - Delta_i x_i B_i (one fused operation);
    h_i carries its own fp32 rounding, so each term mu_i (abar_i h_{i-1}) Delta_i A of the sum has an absolute error of
    up to a few units of eps_fp32 |Delta_i A mu_i h_i|, whatever the size of abar_i h_{i-1} itself.  Per channel p:
        max_n |got - oracle|  <=  tol * max_n |oracle[p, :]|  +  DALOG_C * eps_fp32 * max_n absq[p, :]
    with absq from the oracle.  The second term is what the difference form may add; it is reported so that a run shows
    how much of it was used."""
    got = np.asarray(got, dtype=np.float64)
    want = ref["dA_log"]
    if want.ndim == 1:
        want = want[:, None]; got = got[:, None]
        absq = ref["absq"].sum(axis=1, keepdims=True)
    else:
        absq = ref["absq"]
    assert np.isfinite(got).all(), f"{what}: non-finite values"
    err = np.abs(got - want).max(axis=1)
    strict = tol * np.abs(want).max(axis=1)
    slack = DALOG_C * EPS32 * absq.max(axis=1)
    bad = err > strict + slack
    assert not bad.any(), (f"{what}: {int(bad.sum())} channel rows out of bound, worst p={int(np.argmax(err - strict - slack))}, "
                           f"err {err[bad].max():.3e}")
    over = np.maximum(err - strict, 0.0) / np.maximum(slack, 1e-300)
    return {"rows": int(len(err)), "rows_needing_slack": int((err > strict).sum()), "max_slack_used": float(over.max())}
