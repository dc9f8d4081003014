"""The gradient call is a pure stream of kernel launches: after one eager call (which sets the
function attributes) it can be captured into a CUDA graph and replayed."""
import pytest
import torch

from paper_2501_00692_b200 import binding as B
from paper_2501_00692_b200 import synth
from paper_2501_00692_b200.build import build_library

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("io,tol", [("f32", 1e-5), ("bf16", 1e-2)])
def test_adjoint_grad_replays_from_a_cuda_graph(io, tol):
    build_library()
    w = synth.custom_workload("graph", 23, 2, 1500, 128, tbar=300, io=io)
    theta = synth.layer_params(w, 0, DEV, slow_decay=True)
    x, dy = synth.activations(w, DEV)
    sh = B.shape_of(x, w.d_state)
    _, gb = B.as_workspace_bytes(sh, w.tbar)
    ws = B.alloc_workspace(gb, DEV)
    eager = B.alloc_grads(sh, DEV)
    B.as_adjoint_grad(sh, theta, x, dy, w.tbar, eager, ws)           # eager: first-call set-up happens here
    assert B.as_check_status(ws) == B.AS_OK
    torch.cuda.synchronize()

    grads = B.alloc_grads(sh, DEV)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            B.as_adjoint_grad(sh, theta, x, dy, w.tbar, grads, ws, stream=side)
    for _ in range(2):                                               # two replays: the graph re-zeroes its outputs
        graph.replay()
    torch.cuda.synchronize()
    assert B.as_check_status(ws) == B.AS_OK
    for k in eager:
        if eager[k] is None:
            continue
        a, b = eager[k].float(), grads[k].float()
        scale = float(a.abs().max())
        assert float((a - b).abs().max()) <= tol * max(scale, 1e-30), k
