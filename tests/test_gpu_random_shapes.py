"""Seeded sweep over odd shapes: sequence lengths around chunk and segment boundaries, windows of every relation to the
segment length (shorter, equal, multiples, longer than the sequence), ragged channel tiles, both structures of A."""
import numpy as np
import pytest
import torch

from oracle import ssm_oracle as O
from paper_2501_00692_b200 import binding as B
from paper_2501_00692_b200 import synth
from paper_2501_00692_b200.build import build_library

from gpu_util import TOL, assert_close, compare_grads, theta_f64

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _cases():
    rng = np.random.default_rng(20250106)
    out = []
    for i in range(28):
        T = int(rng.choice([1, 7, 8, 9, 63, 64, 65, 127, 200, 511, 513, 777, 1024, 1500, 2049]))
        P = int(rng.choice([8, 24, 64, 120, 128, 136, 200, 264]))
        rel = rng.choice(["one", "short", "chunk", "seg", "seg+1", "2seg", "full", "over"])
        tbar = {"one": 1, "short": max(1, T // 7), "chunk": 8, "seg": 64, "seg+1": 65, "2seg": 128, "full": T,
                "over": T + 5}[rel]
        batch = int(rng.choice([1, 2, 3]))
        io = "bf16" if i % 4 == 3 else "f32"
        scalar = bool(i % 5 == 2)
        out.append((i, batch, T, P, int(max(1, tbar)), io, scalar))
    return out


@pytest.mark.parametrize("case", _cases(), ids=lambda c: "n%d-B%d-T%d-P%d-tb%d-%s%s" % (c[0], c[1], c[2], c[3], c[4], c[5], "-scalar" if c[6] else ""))
def test_random_shape(case):
    i, batch, T, P, tbar, io, scalar = case
    build_library()
    w = synth.custom_workload("sweep", 30 + i, batch, T, P, tbar=tbar, io=io)
    theta = dict(synth.layer_params(w, 0, DEV, slow_decay=True))
    x, dy = synth.activations(w, DEV)
    if scalar:
        theta["A_log"] = theta["A_log"][:, 5].contiguous()
    sh = B.shape_of(x, w.d_state, a_scalar=scalar)
    _, gb = B.as_workspace_bytes(sh, tbar)
    ws = B.alloc_workspace(gb, DEV)
    grads = B.alloc_grads(sh, DEV)
    y = torch.empty_like(x)
    B.as_ssm_forward(sh, theta, x, y, ws)
    B.as_adjoint_grad(sh, theta, x, dy, tbar, grads, ws)
    assert B.as_check_status(ws) == B.AS_OK
    th = theta_f64(theta)
    if scalar:
        ref = O.batched(O.scalar_adjoint_grad, th, synth.to_f64(x), synth.to_f64(dy), tbar, w.d_state, tier="block")
    else:
        ref = O.batched(O.adjoint_grad, th, synth.to_f64(x), synth.to_f64(dy), tbar, tier="block")
    # a single token has h_0 = 0 and therefore dA_log = 0 exactly in the oracle; see test_degenerate_and_tiny_shapes
    zf = {"dA_log": float(np.abs(ref["dW_B"]).max())}
    compare_grads(grads, ref, TOL[io], zero_floor=zf)
    assert_close(synth.to_f64(y), ref["y"], TOL[io], "y")
