"""Seeded sweep over odd shapes: sequence lengths around chunk and segment boundaries, windows of every relation to the
segment length (shorter, equal, multiples, longer than the sequence), ragged channel tiles, both structures of A."""
import numpy as np
import pytest
import torch

from oracle import ssm_oracle as O
from paper_2501_00692_b200 import binding as B
from paper_2501_00692_b200 import synth
from paper_2501_00692_b200.build import build_library

from gpu_util import TOL, assert_close, compare_all, oracle_adjoint_with_bound

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
    ref = oracle_adjoint_with_bound(theta, x, dy, tbar, tier="block", channel_block=64,
                                    scalar_states=w.d_state if scalar else None)
    # every gradient as a whole tensor, and dA_log channel by channel (a single token has dA_log = 0 exactly in the
    # oracle; the library's rounding residue must stay inside the row-wise bound)
    compare_all(grads, ref, TOL[io])
    assert_close(synth.to_f64(y), ref["y"], TOL[io], "y")
