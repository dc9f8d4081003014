"""Matmul form of the forward for the scalar structure (Table 1 "Scalar SSM"; what as_ssm_forward runs for bf16 I/O and
d_model % 128 == 0) against the fp64 oracle's recurrence with the rates tied, through the C ABI (needs a B200).

The cases cover chunks that are whole, ragged at the segment end and ragged at the sequence end, segments of several
chunks, the three decay laws, and step sizes large enough that channels leave the factorised form and take the
in-kernel recurrence (alone, and mixed with channels that stay in it)."""
import numpy as np
import pytest
import torch

from oracle import ssm_oracle as O
from paper_2501_00692_b200 import binding as B
from paper_2501_00692_b200 import synth
from paper_2501_00692_b200.build import build_library

from gpu_util import TOL, assert_close, theta_f64
from oracle_parallel import ssm_forward as oracle_forward_parallel

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_library()
    B.lib()


def _run(batch, T, P, slow=False, b_delta_range=None, config=31):
    w = synth.custom_workload("scalar-mm", config, batch, T, P, io="bf16")
    theta = dict(synth.layer_params(w, 0, DEV, slow_decay=slow, b_delta_range=b_delta_range))
    theta["A_log"] = theta["A_log"][:, 5].contiguous()            # [P]: the tied rate
    x, _ = synth.activations(w, DEV)
    sh = B.shape_of(x, w.d_state, a_scalar=True)
    fb, _ = B.as_workspace_bytes(sh, T)
    ws = B.alloc_workspace(fb, DEV)
    y = torch.full_like(x, float("nan"))
    B.as_ssm_forward(sh, theta, x, y, ws)
    torch.cuda.synchronize()
    assert B.as_check_status(ws) == 0
    th = O.untie_scalar_A(theta_f64(theta), w.d_state)
    xs = synth.to_f64(x)
    ref = np.stack([oracle_forward_parallel(th, xs[b]) for b in range(batch)])
    return synth.to_f64(y), ref


@pytest.mark.parametrize("batch,T,P,slow", [(2, 2100, 256, False), (2, 2100, 256, True), (1, 64, 128, False),
                                            (3, 65, 128, False), (2, 10, 128, False), (2, 1000, 384, True)])
def test_single_chunk_segments(batch, T, P, slow):
    y, ref = _run(batch, T, P, slow)
    assert_close(y, ref, TOL["bf16"], "y")


def test_segments_of_several_chunks_with_ragged_tails():
    # 32 (channel tile, batch) pairs leave 27 segments of 224 tokens: three whole chunks and one of 32 tokens each,
    # the last segment ends inside a chunk
    y, ref = _run(4, 6000, 1024)
    assert_close(y, ref, TOL["bf16"], "y")


def test_c5_width_segments_of_six_chunks():
    # 16 channel tiles of the widest workload; segments of 368 tokens = five whole chunks and one of 48
    y, ref = _run(1, 20000, 2048, config=5)
    assert_close(y, ref, TOL["bf16"], "y")


@pytest.mark.parametrize("rng", [(1.0, 3.0), (-3.0, 1.0), (-1.0, 1.0)])
def test_large_steps_take_the_recurrence_per_channel(rng):
    # Delta of order one: |a| times half a chunk's Delta sum passes the exponent bound for most or some channels
    y, ref = _run(2, 1500, 256, b_delta_range=rng, config=32)
    assert_close(y, ref, TOL["bf16"], "y")


def test_other_widths_take_the_scan_kernels():
    # d_model not a multiple of 128 keeps the scan kernels: same oracle, same bar
    y, ref = _run(2, 900, 96)
    assert_close(y, ref, TOL["bf16"], "y")


def test_c3_full_size_sampled_channels():
    """Workload C3 at full size with the rates tied (segments of 888 tokens = 13 whole chunks and one of 56, the launch
    configuration the forward benchmark times): y[:, :, p] against the oracle's scan for 32 sampled channels p."""
    from oracle_parallel import _fwd_block, map_bounded, _scan_gb
    w = synth.WORKLOADS["C3"]
    theta = dict(synth.layer_params(w, 0, DEV))
    theta["A_log"] = theta["A_log"][:, 5].contiguous()
    x, _ = synth.activations(w, DEV)
    sh = B.shape_of(x, w.d_state, a_scalar=True)
    ws = B.alloc_workspace(B.as_workspace_bytes(sh, w.seqlen)[0], DEV)
    y = torch.full_like(x, float("nan"))
    B.as_ssm_forward(sh, theta, x, y, ws)
    torch.cuda.synchronize()
    assert B.as_check_status(ws) == 0
    assert torch.isfinite(y.float()).all()
    rng = np.random.default_rng(3)
    sel = np.unique(np.concatenate([[0, 127, 128, w.d_model - 1], rng.choice(w.d_model, 28, replace=False)]))[:32]
    th = O.untie_scalar_A(theta_f64(theta), w.d_state)
    th_sel = dict(th, W_delta=th["W_delta"][sel], b_delta=th["b_delta"][sel], A_log=th["A_log"][sel])
    for b in range(w.batch):
        _, delta, Bm, Cm, A = O.nets(th_sel, synth.to_f64(x[b]))
        xsel = synth.to_f64(x[b][:, sel])
        jobs = [(delta[:, c:c + 8], xsel[:, c:c + 8], Bm, Cm, A[c:c + 8]) for c in range(0, len(sel), 8)]
        yref = np.concatenate(map_bounded(_fwd_block, jobs, _scan_gb(w.seqlen, 8, w.d_state) / 2), axis=1)
        assert_close(synth.to_f64(y[b][:, sel]), yref, TOL["bf16"], f"y[{b}, :, sel]")
