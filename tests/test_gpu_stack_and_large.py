"""Residual stack (Section 3.2, Prop. 3) and the full-size workloads, CUDA vs oracle (needs a B200)."""
import numpy as np
import pytest
import torch

from oracle import ssm_oracle as O
from paper_2501_00692_b200 import binding as B
from paper_2501_00692_b200 import synth
from paper_2501_00692_b200.build import build_library
from paper_2501_00692_b200.stack import Stack

import oracle_parallel as OP
from gpu_util import TOL, assert_close, bf16_round, compare_grads, errors, gpu_adjoint, gpu_forward, theta_f64

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_library()
    B.lib()


def oracle_layer(theta64, x, g, tbar):
    """One layer, batched, on given inputs (the oracle's functions on worker processes)."""
    return OP.batched_adjoint_grad(theta64, x, g, tbar, tier="block", channel_block=64)


def check_stack(io, K, T, P, tbar, mode, batch=2, config=4, every_layer=False):
    """Runs the stack on the GPU and checks it two ways.
    (1) Strictly, per layer: the oracle gets the very bits the layer's kernels consumed (its normalised input and its
        upstream gradient, both in the I/O dtype), so only that layer's own compute error is measured.
    (2) End to end against the oracle's stack with the same storage format: with bf16 I/O every tensor the stack
        stores or hands from layer to layer is rounded to bf16 in the oracle too (its `store` hook), so that again
        only compute error is measured, at the contract's tolerance."""
    w = synth.custom_workload("stack", config, batch, T, P, layers=K, tbar=tbar, io=io)
    thetas = [synth.layer_params(w, k, DEV, slow_decay=(tbar < T)) for k in range(K)]
    y0, g = synth.activations(w, DEV)
    st = Stack(thetas, w.batch, T, P, dtype=w.torch_dtype, device=DEV, tbar=tbar)
    yK = st.forward(y0)
    rec = {k: None for k in (range(K) if every_layer else (K - 1, K // 2, 0))}
    grads, G0 = st.adjoint_grad(g, mode, record=rec)
    torch.cuda.synchronize()
    assert B.as_check_status(st.ws) == B.AS_OK
    if mode == "paper":
        assert B.as_check_status(st.ws_last) == B.AS_OK
    ths = [theta_f64(t) for t in thetas]
    tol = TOL[io]
    for k, (yh, Gk) in rec.items():
        ref = oracle_layer(ths[k], synth.to_f64(yh), synth.to_f64(Gk), tbar)
        for name in O.PARAM_GRADS:
            assert_close(synth.to_f64(grads[k][name]), ref[name], tol, f"layer {k} {name} (same inputs)")
    store = bf16_round if io == "bf16" else None
    acc, G0all, yKref = None, [], []
    for b in range(w.batch):
        ref, G0ref = OP.stack_grad(ths, synth.to_f64(y0)[b], synth.to_f64(g)[b], tbar, mode, store)
        yKref.append(ref["yK"])
        if acc is None:
            acc = [{k: ref["grads"][i][k].copy() for k in O.PARAM_GRADS} for i in range(K)]
        else:
            for i in range(K):
                for k in O.PARAM_GRADS:
                    acc[i][k] += ref["grads"][i][k]
        G0all.append(G0ref)
    worst = 0.0
    l2, _ = errors(synth.to_f64(yK), np.stack(yKref)); worst = max(worst, l2)
    assert l2 <= tol, ("y_K", l2)
    for i in range(K):
        for k in O.PARAM_GRADS:
            l2, _ = errors(synth.to_f64(grads[i][k]), acc[i][k]); worst = max(worst, l2)
            assert l2 <= tol, (i, k, l2)
    if mode == "chained":
        l2, _ = errors(synth.to_f64(G0), np.stack(G0all)); worst = max(worst, l2)
        assert l2 <= tol, ("G_0", l2)
    print(f"stack {io} K={K} T={T} P={P} tbar={tbar} {mode}: worst end-to-end relative L2 error {worst:.3e}")


@pytest.mark.parametrize("io,K,T,P,tbar", [("f32", 3, 300, 40, 300), ("f32", 3, 300, 40, 50), ("bf16", 24, 1024, 128, 256),
                                           ("bf16", 4, 300, 64, 60)])
@pytest.mark.parametrize("mode", ["chained", "paper"])
def test_stack_gradients(io, K, T, P, tbar, mode):
    check_stack(io, K, T, P, tbar, mode)


def test_c4_width_stack_every_layer():
    """The C4 stack at full width and depth (d_model 768, 24 layers, bf16, chained mode) on a sequence the oracle can
    follow: every layer strictly on the bits it consumed, and all gradients plus G_0 end to end."""
    check_stack("bf16", 24, 4096, 768, 1024, "chained", batch=1, every_layer=True)


@pytest.mark.parametrize("io,K,T,P,tbar,with_dx", [("bf16", 5, 1024, 128, 256, True), ("bf16", 3, 300, 64, 50, False),
                                                    ("f32", 3, 300, 40, 70, True)])
def test_layers_call_equals_single_layer_calls(io, K, T, P, tbar, with_dx):
    """as_adjoint_grad_layers (Prop. 3: all layers of the stack in one launch per phase) gives, layer by layer, what
    as_adjoint_grad gives on that layer's parameters and input with the shared upstream gradient - for token counts
    per layer that are (1024 x 2) and are not (300 x 2) a multiple of the 128-row contraction tile, and for fp32 I/O."""
    w = synth.custom_workload("layers", 6, 2, T, P, layers=K, tbar=tbar, io=io)
    thetas = [synth.layer_params(w, k, DEV, slow_decay=True) for k in range(K)]
    _, g = synth.activations(w, DEV)
    xs = torch.stack([synth.activations(synth.custom_workload("layers", 60 + k, 2, T, P, tbar=tbar, io=io), DEV)[0]
                      for k in range(K)]).contiguous()
    sh = B.shape_of(g)
    stacked = {k: torch.stack([th[k] for th in thetas]).contiguous() for k in thetas[0]}
    ws = B.alloc_workspace(B.as_workspace_bytes_layers(sh, K, tbar), DEV)
    gl = B.alloc_grads_layers(sh, K, DEV, with_dx=with_dx)
    B.as_adjoint_grad_layers(sh, K, stacked, xs, g, tbar, gl, ws)
    assert B.as_check_status(ws) == B.AS_OK
    torch.cuda.synchronize()
    for k in range(K):
        one = gpu_adjoint(w, thetas[k], xs[k].contiguous(), g, tbar, with_dx=with_dx)
        ref = OP.batched_adjoint_grad(theta_f64(thetas[k]), synth.to_f64(xs[k]), synth.to_f64(g), tbar, tier="block",
                                      channel_block=64)
        for name in O.PARAM_GRADS + (("dx",) if with_dx else ()):
            a, b_ = synth.to_f64(gl[name][k]), synth.to_f64(one[name])
            assert np.abs(a - b_).max() <= 1e-5 * np.abs(b_).max() + 1e-30, (k, name)   # same kernels, other atomic order
            assert_close(a, ref[name], TOL[io], f"layer {k} {name}")


def test_packed_weights_handle_changes_nothing():
    w = synth.custom_workload("wcat", 7, 2, 900, 96, tbar=200, io="bf16")
    theta = synth.layer_params(w, 0, DEV)
    x, dy = synth.activations(w, DEV)
    sh = B.shape_of(x)
    a = gpu_adjoint(w, theta, x, dy, w.tbar)
    n0 = B.as_launch_count(reset=True)
    gpu_adjoint(w, theta, x, dy, w.tbar)
    with_pack = B.as_launch_count(reset=True)
    th2 = dict(theta)
    th2["Wcat"] = torch.empty(B.as_wcat_bytes(sh), dtype=torch.uint8, device=DEV)
    B.as_pack_weights(sh, 1, theta, th2["Wcat"])
    B.as_launch_count(reset=True)
    b = gpu_adjoint(w, th2, x, dy, w.tbar)
    assert B.as_launch_count(reset=True) == with_pack - 1      # the per-call packing kernel is gone
    for k in O.PARAM_GRADS + ("dx",):
        assert torch.equal(a[k], b[k]) or float((a[k].float() - b[k].float()).abs().max()) <= 1e-5 * float(a[k].float().abs().max()), k


def oracle_batched(theta, x, dy, tbar, channel_block=64):
    return OP.batched_adjoint_grad(theta_f64(theta), synth.to_f64(x), synth.to_f64(dy), tbar, tier="block",
                                   channel_block=channel_block)


def test_c3_full_size_bf16():
    """Workload C3 in the launch configuration the benchmark times, every output against the oracle."""
    w = synth.WORKLOADS["C3"]
    for slow in (False, True):
        theta = synth.layer_params(w, 0, DEV, slow_decay=slow)
        x, dy = synth.activations(w, DEV)
        g = gpu_adjoint(w, theta, x, dy, w.tbar)
        ref = oracle_batched(theta, x, dy, w.tbar)
        compare_grads(g, ref, TOL["bf16"])
        if not slow:
            y = gpu_forward(w, theta, x)
            assert_close(synth.to_f64(y), ref["y"], TOL["bf16"], "y")
        del g, ref
        torch.cuda.empty_cache()


def test_c5_width_full_tensor_bf16():
    """d_model 2,048 (the C5 layer width: the tensor-core contractions run their tail tiles at 2,080 columns) at
    Bsz 1, T = 131,072, Tbar = 4,096, slow-decay law: every output of the forward and of the gradient call against
    the oracle, element by element."""
    w = synth.custom_workload("C5w", 5, 1, 131072, 2048, tbar=4096, io="bf16")
    theta = synth.layer_params(w, 0, DEV, slow_decay=True)
    x, dy = synth.activations(w, DEV)
    g = gpu_adjoint(w, theta, x, dy, w.tbar)
    y = gpu_forward(w, theta, x)
    ref = oracle_batched(theta, x, dy, w.tbar, channel_block=128)
    res = compare_grads(g, ref, TOL["bf16"])
    res["y"] = assert_close(synth.to_f64(y), ref["y"], TOL["bf16"], "y")
    print("C5-width full tensor (rel-L2, rel-max):", {k: (f"{a:.2e}", f"{b:.2e}") for k, (a, b) in res.items()})


def test_c4_full_size_runs_and_matches_on_sampled_layers():
    """Workload C4 (24 layers, T = 32,768, both batch elements) at full size in chained mode: every gradient finite,
    and layers 0, K/2 and K-1 strictly against the oracle on the very bits each consumed (its normalised input and its
    upstream gradient, recorded from the run)."""
    w = synth.WORKLOADS["C4"]
    K = w.layers
    thetas = [synth.layer_params(w, k, DEV) for k in range(K)]
    y0, g = synth.activations(w, DEV)
    st = Stack(thetas, w.batch, w.seqlen, w.d_model, dtype=w.torch_dtype, device=DEV, tbar=w.tbar)
    st.forward(y0)
    rec = {0: None, K // 2: None, K - 1: None}
    grads, G0 = st.adjoint_grad(g, "chained", record=rec)
    torch.cuda.synchronize()
    assert B.as_check_status(st.ws) == B.AS_OK
    for i in range(K):
        for k in O.PARAM_GRADS:
            assert torch.isfinite(grads[i][k]).all(), (i, k)
    assert torch.isfinite(G0.float()).all()
    for k, (yh, Gk) in rec.items():
        ref = oracle_batched(thetas[k], yh, Gk, w.tbar)
        for name in O.PARAM_GRADS:
            assert_close(synth.to_f64(grads[k][name]), ref[name], TOL["bf16"], f"layer {k} {name} (same inputs)")


@pytest.mark.parametrize("slow", [True, False])
def test_c5_full_size_sampled_channels(slow):
    """Workload C5 (T = 2^20, d_model 2048), both decay laws: inputs generated on the device, run at full size, and the
    outputs that depend on a single channel's scan (y[:, p], dA_log[p], db_delta[p], dW_delta[p, :]) checked against
    the oracle for 64 sampled channels p (the oracle reads the device-generated bits back).  The outputs that sum over
    all channels (dx, dW_B, dW_C) are covered at this width by test_c5_width_full_tensor_bf16."""
    w = synth.WORKLOADS["C5"]
    theta = synth.layer_params(w, 0, DEV, slow_decay=slow)
    x, dy = synth.activations(w, DEV)
    g = gpu_adjoint(w, theta, x, dy, w.tbar, with_dx=True)
    y = gpu_forward(w, theta, x)
    for k in O.PARAM_GRADS + ("dx",):
        assert torch.isfinite(g[k].float()).all(), k
    rng = np.random.default_rng(5)
    sel = np.unique(np.concatenate([[0, 127, 128, 2047], rng.choice(w.d_model, 60, replace=False)]))[:64]
    th = theta_f64(theta)
    # a layer whose Delta-net keeps only the sampled rows: the oracle's nets() then yields u, Delta for those channels
    # and the full B_t, C_t; x restricted to those channels feeds the scan.  Done in time pieces (fp64 x is 17 GB).
    T, step = w.seqlen, 1 << 16
    u = np.empty((T, len(sel))); Bm = np.empty((T, w.d_state)); Cm = np.empty((T, w.d_state))
    th_sel = dict(th, W_delta=th["W_delta"][sel], b_delta=th["b_delta"][sel], A_log=th["A_log"][sel])
    for s0 in range(0, T, step):
        u[s0:s0 + step], _, Bm[s0:s0 + step], Cm[s0:s0 + step], _ = O.nets(th_sel, synth.to_f64(x[0, s0:s0 + step]))
    xsel = synth.to_f64(x[0][:, sel]); gs = synth.to_f64(dy[0][:, sel])
    delta = O.softplus(u)
    A = -np.exp(th["A_log"][sel])
    jobs = [(delta[:, c:c + 16], xsel[:, c:c + 16], u[:, c:c + 16], gs[:, c:c + 16], Bm, Cm, A[c:c + 16], w.tbar,
             "block", ()) for c in range(0, len(sel), 16)]
    res = OP.map_bounded(OP._block, jobs, OP._scan_gb(T, 16, w.d_state))
    yref = np.concatenate([r["y"] for r in res], axis=1)
    du = np.concatenate([r["du"] for r in res], axis=1)
    dAl = np.concatenate([r["dA_log"] for r in res], axis=0)
    dWd = np.zeros((len(sel), w.d_model))
    for s0 in range(0, T, step):
        dWd += du[s0:s0 + step].T @ synth.to_f64(x[0, s0:s0 + step])
    tol = TOL["bf16"]
    assert_close(synth.to_f64(y[0][:, sel]), yref, tol, "y[:, sel]")
    assert_close(synth.to_f64(g["dA_log"][sel]), dAl, tol, "dA_log[sel]")
    assert_close(synth.to_f64(g["db_delta"][sel]), du.sum(axis=0), tol, "db_delta[sel]")
    assert_close(synth.to_f64(g["dW_delta"][sel]), dWd, tol, "dW_delta[sel]")
