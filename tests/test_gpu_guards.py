"""Out-of-bounds write detection without a sanitizer: every output and the scratch buffer sit between guard
regions filled with a pattern; after each entry point the guards must be untouched.  Plus run-to-run agreement."""
import pytest
import torch

from paper_2501_00692_b200 import binding as B
from paper_2501_00692_b200 import synth
from paper_2501_00692_b200.build import build_library

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
GUARD = 4096


def guarded(nbytes):
    """(view of nbytes between two guards, whole buffer)."""
    n = (int(nbytes) + 255) // 256 * 256
    whole = torch.full((n + 2 * GUARD,), 0xA5, dtype=torch.uint8, device=DEV)
    return whole[GUARD:GUARD + n], whole, n


def guards_intact(whole, n):
    return bool((whole[:GUARD] == 0xA5).all()) and bool((whole[GUARD + n:] == 0xA5).all())


def typed(view, shape, dtype):
    numel = 1
    for s in shape:
        numel *= s
    return view[: numel * torch.empty((), dtype=dtype).element_size()].view(dtype).view(*shape)


@pytest.mark.parametrize("io", ["f32", "bf16"])
@pytest.mark.parametrize("batch,T,P,tbar", [(2, 300, 40, 70), (1, 1000, 136, 2000), (2, 5, 8, 2), (1, 2048, 256, 512)])
def test_no_write_outside_buffers(batch, T, P, tbar, io):
    build_library()
    w = synth.custom_workload("guard", 18, batch, T, P, tbar=tbar, io=io)
    theta = synth.layer_params(w, 0, DEV)
    x, dy = synth.activations(w, DEV)
    sh = B.shape_of(x)
    fb, gb = B.as_workspace_bytes(sh, tbar)
    esz = x.element_size()
    bufs = {}
    ws_v, ws_w, ws_n = guarded(gb)
    N = w.d_state
    shapes = {"dW_delta": (P, P), "db_delta": (P,), "dW_B": (N, P), "dW_C": (N, P), "dA_log": (P, N)}
    grads = {}
    for k, shp in shapes.items():
        numel = 1
        for s in shp:
            numel *= s
        v, wh, n = guarded(numel * 4)
        bufs[k] = (wh, n)
        grads[k] = typed(v, shp, torch.float32)
    v, wh, n = guarded(batch * T * P * esz)
    bufs["dx"] = (wh, n)
    grads["dx"] = typed(v, (batch, T, P), x.dtype)
    v, wh, n = guarded(batch * T * P * esz)
    bufs["y"] = (wh, n)
    y = typed(v, (batch, T, P), x.dtype)

    def check(what):
        torch.cuda.synchronize()
        assert guards_intact(ws_w, ws_n), f"{what}: wrote outside the workspace"
        for k, (wh_, n_) in bufs.items():
            assert guards_intact(wh_, n_), f"{what}: wrote outside {k}"

    B.as_ssm_forward(sh, theta, x, y, ws_v); check("as_ssm_forward")
    B.as_adjoint_grad(sh, theta, x, dy, tbar, grads, ws_v); check("as_adjoint_grad")
    first = {k: v.clone() for k, v in grads.items()}
    B.as_adjoint_grad(sh, theta, x, dy, tbar, grads, ws_v); check("as_adjoint_grad (second call)")
    # run-to-run: atomics make bitwise equality a non-promise, but the two runs must agree to rounding (with bf16
    # I/O a different summation order can flip the bf16 rounding of an intermediate or an output element)
    rtol = 1e-5 if io == "f32" else 1e-2
    for k in grads:
        a, b = first[k].double(), grads[k].double()
        assert float((a - b).abs().max()) <= rtol * float(a.abs().max()) + 1e-30, k
    B.as_adjoint_grad(sh, theta, x, dy, T, grads, ws_v); check("as_adjoint_grad (full)")
    B.as_full_bptt_grad(sh, theta, x, dy, grads, ws_v); check("as_full_bptt_grad")
    yh = torch.empty_like(x)
    B.as_rmsnorm_fwd(sh, x, y); B.as_rmsnorm_bwd_add(sh, x, dy, grads["dx"]); B.as_residual_add(sh, x, dy, y)
    check("glue")
    assert B.as_check_status(ws_v) == 0


def test_bounded_wait_reports_timeout_and_context_survives():
    """A device-side wait that can never be satisfied gives up after its poll limit, the host reads AS_ERR_TIMEOUT
    from the status word, and the next call on the same context works and reports AS_OK."""
    build_library()
    ws = torch.zeros(4096, dtype=torch.uint8, device=DEV)
    B.as_wait_selftest(ws, poll_limit=2048)
    assert B.as_check_status(ws) == B.AS_ERR_TIMEOUT
    w = synth.custom_workload("after", 19, 1, 64, 32, io="f32")
    theta = synth.layer_params(w, 0, DEV)
    x, _ = synth.activations(w, DEV)
    sh = B.shape_of(x)
    fb, _ = B.as_workspace_bytes(sh, 64)
    ws2 = B.alloc_workspace(fb, DEV)
    y = torch.empty_like(x)
    B.as_ssm_forward(sh, theta, x, y, ws2)
    assert B.as_check_status(ws2) == B.AS_OK
    assert torch.isfinite(y).all()
