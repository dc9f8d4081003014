"""CUDA path vs the fp64 oracle, element by element, through the C ABI (needs a B200)."""
import numpy as np
import pytest
import torch

from oracle import ssm_oracle as O
from paper_2501_00692_b200 import binding as B
from paper_2501_00692_b200 import synth
from paper_2501_00692_b200.build import build_library

from gpu_util import (TOL, assert_close, assert_dalog_rows, compare_all, compare_grads, gpu_adjoint, gpu_forward,
                      oracle_adjoint, oracle_adjoint_with_bound, theta_f64)

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_library()
    B.lib()


def setup(w, slow=False, layer=0):
    theta = synth.layer_params(w, layer, DEV, slow_decay=slow)
    x, dy = synth.activations(w, DEV)
    return theta, x, dy


def test_c1_forward_and_full_adjoint_fp32():
    w = synth.WORKLOADS["C1"]
    theta, x, dy = setup(w)
    y = gpu_forward(w, theta, x)
    yref = np.stack([O.ssm_forward(theta_f64(theta), synth.to_f64(x)[b]) for b in range(w.batch)])
    assert_close(synth.to_f64(y), yref, TOL["f32"], "y")
    ref = oracle_adjoint(theta, x, dy, w.tbar, tier="direct")
    compare_grads(gpu_adjoint(w, theta, x, dy, w.tbar), ref, TOL["f32"])
    # truncated == full once the window covers the sequence (Eq. 7), on the GPU too
    compare_grads(gpu_adjoint(w, theta, x, dy, w.seqlen + 5), ref, TOL["f32"])


def test_c1_bptt_comparator_matches_oracle_and_adjoint():
    w = synth.WORKLOADS["C1"]
    theta, x, dy = setup(w)
    th = theta_f64(theta)
    ref = O.batched(O.bptt_grad, th, synth.to_f64(x), synth.to_f64(dy))
    gb = gpu_adjoint(w, theta, x, dy, w.tbar, bptt=True)
    compare_grads(gb, ref, TOL["f32"])
    ga = gpu_adjoint(w, theta, x, dy, w.tbar)
    for k in O.PARAM_GRADS + ("dx",):
        assert_close(synth.to_f64(ga[k]), synth.to_f64(gb[k]), TOL["f32"], "adjoint vs bptt " + k)


@pytest.mark.parametrize("slow", [False, True])
@pytest.mark.parametrize("tbar", [1, 2, 7, 8, 9, 63, 64, 65, 127, 128, 129, 200, 299, 300, 301])
def test_ragged_small_shapes_window_edges(tbar, slow):
    # several 64-token segments with a ragged last one, d_model not a multiple of the warp width,
    # windows below / at / above segment multiples
    w = synth.custom_workload("ragged", 11, 2, 300, 40, tbar=tbar, io="f32")
    theta, x, dy = setup(w, slow)
    ref = oracle_adjoint(theta, x, dy, tbar, tier="direct")
    compare_grads(gpu_adjoint(w, theta, x, dy, tbar), ref, TOL["f32"])


def test_impulse_window_edges_on_gpu():
    # upstream gradient = one impulse: B-path outputs are non-zero exactly on the window (Eq. 7 ranges)
    w = synth.custom_workload("impulse", 12, 1, 200, 32, tbar=70, io="f32")
    theta, x, dy = setup(w, slow=True)
    dy.zero_()
    tp, pp = 150, 5
    dy[0, tp, pp] = 1.0
    g = gpu_adjoint(w, theta, x, dy, w.tbar)
    ref = oracle_adjoint(theta, x, dy, w.tbar, tier="direct")
    compare_grads(g, ref, TOL["f32"])
    # dx = dx_dir + (dense parts): rows inside the window carry signal, rows after the impulse are exactly
    # zero, rows before the window hold only the rounding residue of the exact window-exit subtraction
    dx = np.abs(synth.to_f64(g["dx"])[0]).max(axis=1)
    lo = tp - w.tbar + 1
    assert (dx[tp + 1:] == 0).all()
    assert (dx[lo:tp + 1] > 1e-3 * dx.max()).all()
    assert (dx[:lo] < 1e-5 * dx.max()).all()


def test_accumulate_flag_and_no_dx():
    w = synth.custom_workload("acc", 13, 1, 128, 32, tbar=20, io="f32")
    theta, x, dy = setup(w)
    g1 = gpu_adjoint(w, theta, x, dy, w.tbar)
    g2 = gpu_adjoint(w, theta, x, dy, w.tbar, with_dx=False)
    g2 = gpu_adjoint(w, theta, x, dy, w.tbar, flags=B.AS_ACCUMULATE, grads=g2, with_dx=False)
    for k in O.PARAM_GRADS:
        assert_close(synth.to_f64(g2[k]), 2 * synth.to_f64(g1[k]), 1e-5, k)


def test_c2_truncated_and_full_fp32():
    w = synth.WORKLOADS["C2"]
    for slow in (False, True):
        theta, x, dy = setup(w, slow)
        ref = oracle_adjoint(theta, x, dy, w.tbar, tier="direct")       # Tbar = 64: the defining double sum
        compare_grads(gpu_adjoint(w, theta, x, dy, w.tbar), ref, TOL["f32"])
        full = oracle_adjoint(theta, x, dy, w.seqlen, tier="block")
        compare_grads(gpu_adjoint(w, theta, x, dy, w.seqlen), full, TOL["f32"])
        if slow:   # the window is visible: truncated and full differ by far more than the tolerance
            assert np.abs(ref["dW_B"] - full["dW_B"]).max() / np.abs(full["dW_B"]).max() > 1e-2


@pytest.mark.parametrize("slow", [False, True])
def test_bf16_multi_segment(slow):
    w = synth.custom_workload("bf16", 14, 2, 4096, 128, tbar=1000, io="bf16")
    theta, x, dy = setup(w, slow)
    ref = oracle_adjoint(theta, x, dy, w.tbar, tier="block")
    compare_grads(gpu_adjoint(w, theta, x, dy, w.tbar), ref, TOL["bf16"])
    y = gpu_forward(w, theta, x)
    assert_close(synth.to_f64(y), ref["y"], TOL["bf16"], "y")


def test_rmsnorm_glue():
    w = synth.custom_workload("norm", 15, 2, 33, 72, io="f32")
    _, y, d = setup(w)
    sh = B.shape_of(y)
    yhat = torch.empty_like(y)
    B.as_rmsnorm_fwd(sh, y, yhat)
    assert_close(synth.to_f64(yhat), O.rmsnorm(synth.to_f64(y)), 1e-5, "rmsnorm")
    G = d.clone()
    B.as_rmsnorm_bwd_add(sh, y, d, G)
    assert_close(synth.to_f64(G), synth.to_f64(d) + O.rmsnorm_vjp(synth.to_f64(y), synth.to_f64(d)), 1e-5, "rmsnorm vjp")
    out = torch.empty_like(y)
    B.as_residual_add(sh, y, d, out)
    assert torch.equal(out, y + d)


@pytest.mark.parametrize("io", ["f32", "bf16"])
@pytest.mark.parametrize("batch,T,P,tbar", [(1, 1, 8, 1), (3, 5, 8, 2), (2, 7, 24, 100), (1, 9, 136, 3), (2, 64, 264, 64),
                                            (1, 65, 40, 1)])
def test_degenerate_and_tiny_shapes(batch, T, P, tbar, io):
    # sequences shorter than one chunk, one token, the narrowest d_model, widths that leave a ragged channel tile,
    # bf16 widths that take the FP32-pipe contraction path (d_model not a multiple of 32)
    w = synth.custom_workload("tiny", 16, batch, T, P, tbar=tbar, io=io)
    theta, x, dy = setup(w, slow=True)
    ref = oracle_adjoint_with_bound(theta, x, dy, tbar, tier="direct")
    # With a single token dA_log is identically zero in the oracle (h_0 = 0); the library's value is then pure
    # rounding of h_1 - Delta_1 x_1 B_1 and must stay inside the row-wise bound built from the oracle's own mu and h.
    compare_all(gpu_adjoint(w, theta, x, dy, tbar), ref, TOL[io])
    y = gpu_forward(w, theta, x)
    assert_close(synth.to_f64(y), ref["y"], TOL[io], "y")
    gb = gpu_adjoint(w, theta, x, dy, T, bptt=True)
    compare_grads(gb, oracle_adjoint(theta, x, dy, T, tier="direct"), TOL[io])


@pytest.mark.parametrize("io", ["f32", "bf16"])
@pytest.mark.parametrize("law", ["fast", "standard", "slow"])
@pytest.mark.parametrize("T", [2, 3, 8, 64, 300])
def test_dalog_row_by_row(T, law, io):
    """dA_log channel by channel where abar_i h_{i-1} is small against h_i: very short sequences (h_{i-1} is zero or
    one step old) and the fast-decay corner b_delta ~ U(-1, 1) (abar << 1).  The library forms abar_i h_{i-1} as
    h_i - Delta_i x_i B_i; the bound allows DALOG_C rounding units of h_i per term beyond the tolerance and the test
    reports how much of that allowance was used."""
    w = synth.custom_workload("dalog", 18, 2, T, 72, tbar=max(1, T // 2), io=io)
    rng = {"fast": (-1.0, 1.0), "standard": None, "slow": (-9.0, -7.0)}[law]
    theta = synth.layer_params(w, 0, DEV, b_delta_range=rng)
    x, dy = synth.activations(w, DEV)
    for tbar in (w.tbar, T):
        ref = oracle_adjoint_with_bound(theta, x, dy, tbar, tier="direct")
        g = gpu_adjoint(w, theta, x, dy, tbar)
        use = assert_dalog_rows(synth.to_f64(g["dA_log"]), ref, TOL[io])
        compare_grads(g, ref, TOL[io], keys=("dW_delta", "db_delta", "dW_B", "dW_C", "dx"))
        print(f"dA_log rows T={T} law={law} io={io} tbar={tbar}: {use}")


def test_bptt_comparator_bf16_multi_segment():
    """as_full_bptt_grad on bf16 I/O over several of its 64-token checkpoint segments and time segments."""
    w = synth.custom_workload("bptt16", 19, 2, 4100, 160, io="bf16")
    theta, x, dy = setup(w, slow=True)
    ref = O.batched(O.bptt_grad, theta_f64(theta), synth.to_f64(x), synth.to_f64(dy))
    gb = gpu_adjoint(w, theta, x, dy, w.seqlen, bptt=True)
    compare_grads(gb, ref, TOL["bf16"])
    ga = gpu_adjoint(w, theta, x, dy, w.seqlen)
    compare_grads(ga, ref, TOL["bf16"])


def test_zero_upstream_gradient_gives_zero():
    w = synth.custom_workload("zero", 17, 1, 200, 64, tbar=50, io="f32")
    theta, x, dy = setup(w)
    dy.zero_()
    g = gpu_adjoint(w, theta, x, dy, w.tbar)
    for k in O.PARAM_GRADS + ("dx",):
        assert float(g[k].abs().max()) == 0.0, k


# ---- scalar structure: one decay rate per channel (Table 1 "Scalar SSM") ---------------------------------------------
@pytest.mark.parametrize("io,T,P,tbar", [("f32", 700, 64, 700), ("f32", 1300, 136, 90), ("bf16", 2100, 256, 300),
                                         ("bf16", 900, 96, 900)])
def test_scalar_structure_matches_oracle(io, T, P, tbar):
    w = synth.custom_workload("scalar", 21, 2, T, P, tbar=tbar, io=io)
    theta, x, dy = setup(w, slow=True)
    theta = dict(theta)
    theta["A_log"] = theta["A_log"][:, 3].contiguous()            # [P]: the tied rate
    sh = B.shape_of(x, w.d_state, a_scalar=True)
    fb, gb = B.as_workspace_bytes(sh, tbar)
    ws = B.alloc_workspace(gb, DEV)
    grads = B.alloc_grads(sh, DEV)
    assert tuple(grads["dA_log"].shape) == (P,)
    y = torch.empty_like(x)
    B.as_ssm_forward(sh, theta, x, y, ws)
    B.as_adjoint_grad(sh, theta, x, dy, tbar, grads, ws)
    assert B.as_check_status(ws) == 0
    th = theta_f64(theta)
    ref = O.batched(O.scalar_adjoint_grad, th, synth.to_f64(x), synth.to_f64(dy), tbar, w.d_state, tier="block")
    compare_grads(grads, ref, TOL[io])
    assert_close(synth.to_f64(y), ref["y"], TOL[io], "y")
    if tbar >= T:   # the backpropagation comparator ties the rate the same way
        gb2 = B.alloc_grads(sh, DEV)
        B.as_full_bptt_grad(sh, theta, x, dy, gb2, ws)
        compare_grads(gb2, ref, TOL[io])
