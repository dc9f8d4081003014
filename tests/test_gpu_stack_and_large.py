"""Residual stack (Section 3.2, Prop. 3) and the full-size workloads, CUDA vs oracle (needs a B200)."""
import numpy as np
import pytest
import torch

from oracle import ssm_oracle as O
from paper_2501_00692_b200 import binding as B
from paper_2501_00692_b200 import synth
from paper_2501_00692_b200.build import build_library
from paper_2501_00692_b200.stack import Stack

from gpu_util import TOL, assert_close, compare_grads, gpu_adjoint, gpu_forward, oracle_adjoint, theta_f64

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_library()
    B.lib()


@pytest.mark.parametrize("io,K,T,P,tbar", [("f32", 3, 300, 40, 300), ("f32", 3, 300, 40, 50), ("bf16", 24, 1024, 128, 256)])
@pytest.mark.parametrize("mode", ["chained", "paper"])
def test_stack_gradients(io, K, T, P, tbar, mode):
    w = synth.custom_workload("stack", 4, 2, T, P, layers=K, tbar=tbar, io=io)
    thetas = [synth.layer_params(w, k, DEV, slow_decay=(tbar < T)) for k in range(K)]
    y0, g = synth.activations(w, DEV)
    st = Stack(thetas, w.batch, T, P, dtype=w.torch_dtype, device=DEV, tbar=tbar)
    yK = st.forward(y0)
    rec = {K - 1: None, K // 2: None, 0: None}
    grads, G0 = st.adjoint_grad(g, mode, record=rec)
    torch.cuda.synchronize()
    ths = [theta_f64(t) for t in thetas]
    tol = TOL[io]
    # (1) strict, per layer: the oracle gets the very bits the layer's kernels consumed (its normalised input and its
    #     upstream gradient, both in the I/O dtype), so only the layer's own compute error is measured
    for k, (yh, Gk) in rec.items():
        ref = O.batched(O.adjoint_grad, ths[k], synth.to_f64(yh), synth.to_f64(Gk), tbar, tier="block")
        for name in O.PARAM_GRADS:
            assert_close(synth.to_f64(grads[k][name]), ref[name], tol, f"layer {k} {name} (same inputs)")
    # (2) end to end against the fp64 stack.  With bf16 storage every one of the K intermediate activations (and, in
    #     chained mode, gradients) is rounded to 2^-9 on the GPU but not in the oracle, so the bar is on the relative
    #     L2 error only and widened by sqrt(K) roundings.
    e2e = tol if io == "f32" else tol * max(1.0, np.sqrt(K) / 2)
    acc, G0all = None, []
    for b in range(w.batch):
        ref, G0ref = O.stack_grad(ths, synth.to_f64(y0)[b], synth.to_f64(g)[b], tbar, mode=mode, tier="block")
        if acc is None:
            acc = [{k: ref[i][k].copy() for k in O.PARAM_GRADS} for i in range(K)]
        else:
            for i in range(K):
                for k in O.PARAM_GRADS:
                    acc[i][k] += ref[i][k]
        G0all.append(G0ref)
    from gpu_util import errors
    ys, _ = O.stack_forward(ths, synth.to_f64(y0)[0])
    assert errors(synth.to_f64(yK)[0], ys[-1])[0] <= e2e
    for i in range(K):
        for k in O.PARAM_GRADS:
            l2, _ = errors(synth.to_f64(grads[i][k]), acc[i][k])
            assert l2 <= e2e, (i, k, l2)
    if mode == "chained":
        assert errors(synth.to_f64(G0), np.stack(G0all))[0] <= e2e


def test_paper_mode_on_two_streams_equals_one_stream():
    """Prop. 3's layers are independent: spreading them over two streams (each with its own workspace) changes nothing
    but the order of the fp32 atomic sums."""
    K, T, P, tbar = 6, 1200, 128, 256
    w = synth.custom_workload("stack2", 5, 2, T, P, layers=K, tbar=tbar, io="bf16")
    thetas = [synth.layer_params(w, k, DEV, slow_decay=True) for k in range(K)]
    y0, g = synth.activations(w, DEV)
    out = []
    for ns in (1, 2):
        st = Stack(thetas, w.batch, T, P, dtype=w.torch_dtype, device=DEV, tbar=tbar, paper_streams=ns)
        st.forward(y0)
        grads, _ = st.adjoint_grad(g, "paper")
        torch.cuda.synchronize()
        assert B.as_check_status(st.ws) == B.AS_OK
        out.append(grads)
    for a, b in zip(*out):
        for k in O.PARAM_GRADS:
            scale = float(a[k].abs().max())
            assert float((a[k] - b[k]).abs().max()) <= 1e-2 * scale, k


def test_c3_full_size_bf16():
    """Workload C3 in the launch configuration the benchmark times, every output against the oracle."""
    w = synth.WORKLOADS["C3"]
    for slow in (False, True):
        theta = synth.layer_params(w, 0, DEV, slow_decay=slow)
        x, dy = synth.activations(w, DEV)
        g = gpu_adjoint(w, theta, x, dy, w.tbar)
        ref = oracle_adjoint(theta, x, dy, w.tbar, tier="block", channel_block=192)
        compare_grads(g, ref, TOL["bf16"])
        if not slow:
            y = gpu_forward(w, theta, x)
            assert_close(synth.to_f64(y), ref["y"], TOL["bf16"], "y")
        del g, ref
        torch.cuda.empty_cache()


def test_c4_full_size_runs_and_matches_on_sampled_layers():
    """Workload C4 (24 layers, T=32768): run at full size; the top layer's gradients in paper mode depend only on
    that layer's stored input, so they are checked against the oracle on that input (read back from the GPU)."""
    w = synth.WORKLOADS["C4"]
    thetas = [synth.layer_params(w, k, DEV) for k in range(w.layers)]
    y0, g = synth.activations(w, DEV)
    st = Stack(thetas, w.batch, w.seqlen, w.d_model, dtype=w.torch_dtype, device=DEV, tbar=w.tbar)
    st.forward(y0)
    grads, G0 = st.adjoint_grad(g, "chained")
    torch.cuda.synchronize()
    for i in range(w.layers):
        for k in O.PARAM_GRADS:
            assert torch.isfinite(grads[i][k]).all(), (i, k)
    assert torch.isfinite(G0.float()).all()
    # top layer, chained == paper mode there: oracle on the GPU's own normalised input (bf16 bits read back)
    k = w.layers - 1
    yhat = torch.empty_like(y0)
    B.as_rmsnorm_fwd(st.shape, st.ys[k], yhat)
    ref = oracle_adjoint(thetas[k], yhat[:1], g[:1], w.tbar, tier="block", channel_block=192)
    g1 = gpu_adjoint(synth.custom_workload("c4top", 4, 1, w.seqlen, w.d_model, tbar=w.tbar, io="bf16"), thetas[k],
                     yhat[:1].contiguous(), g[:1].contiguous(), w.tbar)
    compare_grads(g1, ref, TOL["bf16"])


def test_c5_full_size_sampled_channels():
    """Workload C5 (T = 2^20, d_model 2048): inputs generated on the device, run at full size, and the outputs that
    depend on a single channel's scan (y[:, p], dA_log[p], db_delta[p], dW_delta[p, :]) are checked against the
    oracle for sampled channels p (the oracle reads the device-generated bits back)."""
    w = synth.WORKLOADS["C5"]
    theta = synth.layer_params(w, 0, DEV, slow_decay=True)
    x, dy = synth.activations(w, DEV)
    g = gpu_adjoint(w, theta, x, dy, w.tbar, with_dx=True)
    y = gpu_forward(w, theta, x)
    for k in O.PARAM_GRADS + ("dx",):
        assert torch.isfinite(g[k].float()).all(), k
    sel = [3, 700, 1111, 2047]
    th = theta_f64(theta)
    T, step = w.seqlen, 1 << 16
    u = np.empty((T, len(sel))); Bm = np.empty((T, w.d_state)); Cm = np.empty((T, w.d_state))
    for s0 in range(0, T, step):      # chunked fp64 widening of x: the full array would be 17 GB
        xc = synth.to_f64(x[0, s0:s0 + step])
        u[s0:s0 + step] = xc @ th["W_delta"][sel].T + th["b_delta"][sel]
        Bm[s0:s0 + step] = xc @ th["W_B"].T
        Cm[s0:s0 + step] = xc @ th["W_C"].T
    xsel = synth.to_f64(x[0][:, sel]); gs = synth.to_f64(dy[0][:, sel])
    delta = O.softplus(u)
    A = -np.exp(th["A_log"][sel])
    yref, H, abar = O.scan_forward(delta, xsel, Bm, Cm, A)
    mu = O.mu_block(abar, gs, Cm, w.tbar)
    tok = O.token_cotangents(mu, H, abar, gs, delta, xsel, u, Bm, A)
    dWd = np.zeros((len(sel), w.d_model))
    for s0 in range(0, T, step):
        dWd += tok["du"][s0:s0 + step].T @ synth.to_f64(x[0, s0:s0 + step])
    tol = TOL["bf16"]
    assert_close(synth.to_f64(y[0][:, sel]), yref, tol, "y[:, sel]")
    assert_close(synth.to_f64(g["dA_log"][sel]), tok["dA_log"], tol, "dA_log[sel]")
    assert_close(synth.to_f64(g["db_delta"][sel]), tok["du"].sum(axis=0), tol, "db_delta[sel]")
    assert_close(synth.to_f64(g["dW_delta"][sel]), dWd, tol, "dW_delta[sel]")
