"""ctypes binding of libadjoint_ssm.so: the same entry points as include/adjoint_ssm.h.

Argument marshalling only - torch tensors supply device pointers and the current stream; every step
of the computation runs inside the library's kernels.  There is no fallback: if the library has not
been built (``python -m paper_2501_00692_b200.build``), the first call raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libadjoint_ssm.so")

AS_F32, AS_BF16 = 0, 1
AS_A_DIAGONAL, AS_A_SCALAR = 0, 1
AS_ACCUMULATE = 1
AS_OK = 0
AS_ERR_NULL, AS_ERR_SHAPE, AS_ERR_DTYPE, AS_ERR_TBAR = -1, -2, -3, -4
AS_ERR_WORKSPACE, AS_ERR_ALIGN, AS_ERR_CUDA, AS_ERR_TIMEOUT, AS_ERR_LIMIT = -5, -6, -7, -8, -9

EXPORTS = ("as_version", "as_strerror", "as_workspace_bytes", "as_check_status", "as_ssm_forward",
           "as_adjoint_grad", "as_full_bptt_grad", "as_rmsnorm_fwd", "as_residual_add", "as_rmsnorm_bwd_add",
           "as_launch_count", "as_set_timing", "as_get_timing", "as_ssm_forward_static", "as_wait_selftest", "as_sm_count",
           "as_adjoint_grad_layers", "as_workspace_bytes_layers", "as_wcat_bytes", "as_pack_weights")
AS_STATIC_SCRATCH_BYTES = 32 << 20
AS_NUM_PHASES = 6
PHASES = ("projections", "prepass", "fixup", "adjoint_main", "weight_grads", "input_grad")


class as_shape_t(C.Structure):
    _fields_ = [("batch", C.c_int32), ("seqlen", C.c_int64), ("d_model", C.c_int32),
                ("d_state", C.c_int32), ("io", C.c_int32), ("a_structure", C.c_int32)]


class as_params_t(C.Structure):
    _fields_ = [("W_delta", C.c_void_p), ("b_delta", C.c_void_p), ("W_B", C.c_void_p),
                ("W_C", C.c_void_p), ("A_log", C.c_void_p), ("Wcat", C.c_void_p)]


class as_grads_t(C.Structure):
    _fields_ = [("dW_delta", C.c_void_p), ("db_delta", C.c_void_p), ("dW_B", C.c_void_p),
                ("dW_C", C.c_void_p), ("dA_log", C.c_void_p), ("dx", C.c_void_p)]


class AsError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} ({code})")


_lib = None


def lib() -> C.CDLL:
    """The loaded shared library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} not found: build it with `python -m paper_2501_00692_b200.build` "
                               "(there is no CPU or PyTorch fallback)")
        L = C.CDLL(LIB_PATH)
        L.as_version.restype = C.c_int
        L.as_strerror.restype = C.c_char_p
        L.as_strerror.argtypes = [C.c_int]
        L.as_workspace_bytes.argtypes = [C.POINTER(as_shape_t), C.c_int64, C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]
        L.as_check_status.argtypes = [C.c_void_p, C.c_void_p]
        L.as_ssm_forward.argtypes = [C.POINTER(as_shape_t), C.POINTER(as_params_t), C.c_void_p, C.c_void_p,
                                     C.c_void_p, C.c_size_t, C.c_void_p]
        L.as_adjoint_grad.argtypes = [C.POINTER(as_shape_t), C.POINTER(as_params_t), C.c_void_p, C.c_void_p,
                                      C.c_int64, C.c_uint32, C.POINTER(as_grads_t), C.c_void_p, C.c_size_t, C.c_void_p]
        L.as_full_bptt_grad.argtypes = [C.POINTER(as_shape_t), C.POINTER(as_params_t), C.c_void_p, C.c_void_p,
                                        C.c_uint32, C.POINTER(as_grads_t), C.c_void_p, C.c_size_t, C.c_void_p]
        L.as_rmsnorm_fwd.argtypes = [C.POINTER(as_shape_t), C.c_void_p, C.c_void_p, C.c_float, C.c_void_p]
        L.as_residual_add.argtypes = [C.POINTER(as_shape_t), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.as_rmsnorm_bwd_add.argtypes = [C.POINTER(as_shape_t), C.c_void_p, C.c_void_p, C.c_void_p, C.c_float,
                                         C.c_void_p]
        L.as_ssm_forward_static.argtypes = [C.POINTER(as_shape_t), C.POINTER(as_params_t), C.c_void_p, C.c_void_p,
                                            C.c_void_p]
        L.as_wait_selftest.argtypes = [C.c_void_p, C.c_size_t, C.c_uint32, C.c_void_p]
        L.as_adjoint_grad_layers.argtypes = [C.POINTER(as_shape_t), C.c_int32, C.POINTER(as_params_t), C.c_void_p,
                                             C.c_void_p, C.c_int64, C.c_uint32, C.POINTER(as_grads_t), C.c_void_p,
                                             C.c_size_t, C.c_void_p]
        L.as_workspace_bytes_layers.argtypes = [C.POINTER(as_shape_t), C.c_int32, C.c_int64, C.POINTER(C.c_size_t)]
        L.as_wcat_bytes.argtypes = [C.POINTER(as_shape_t), C.c_int32]
        L.as_pack_weights.argtypes = [C.POINTER(as_shape_t), C.c_int32, C.POINTER(as_params_t), C.c_void_p, C.c_void_p]
        L.as_launch_count.argtypes = [C.c_int]
        L.as_set_timing.argtypes = [C.c_int]
        L.as_get_timing.argtypes = [C.POINTER(C.c_float), C.c_int]
        for name in EXPORTS:
            if name not in ("as_strerror", "as_launch_count", "as_wcat_bytes"):
                getattr(L, name).restype = C.c_int
        L.as_launch_count.restype = C.c_int64
        L.as_wcat_bytes.restype = C.c_size_t
        _lib = L
    return _lib


# ------------------------------------------------------------------------------------------ marshalling
def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _check(code: int, where: str):
    if code != AS_OK:
        raise AsError(code, where)


def make_shape(batch, seqlen, d_model, d_state=16, io=AS_F32, a_structure=AS_A_DIAGONAL) -> as_shape_t:
    return as_shape_t(int(batch), int(seqlen), int(d_model), int(d_state), int(io), int(a_structure))


def shape_of(x: torch.Tensor, d_state=16, a_scalar=False) -> as_shape_t:
    io = {torch.float32: AS_F32, torch.bfloat16: AS_BF16}[x.dtype]
    return make_shape(x.shape[0], x.shape[1], x.shape[2], d_state, io, AS_A_SCALAR if a_scalar else AS_A_DIAGONAL)


def make_params(theta: dict) -> as_params_t:
    """theta may carry an optional "Wcat" (the packed weights of as_pack_weights)."""
    return as_params_t(*[_ptr(theta[k]) for k in ("W_delta", "b_delta", "W_B", "W_C", "A_log")], _ptr(theta.get("Wcat")))


def alloc_grads(shape: as_shape_t, device, with_dx=True) -> dict:
    """Caller-owned gradient buffers (device memory comes from torch)."""
    P, N = shape.d_model, shape.d_state
    f = dict(dtype=torch.float32, device=device)
    g = {"dW_delta": torch.empty(P, P, **f), "db_delta": torch.empty(P, **f), "dW_B": torch.empty(N, P, **f),
         "dW_C": torch.empty(N, P, **f),
         "dA_log": torch.empty(P, **f) if shape.a_structure != AS_A_DIAGONAL else torch.empty(P, N, **f), "dx": None}
    if with_dx:
        dt = torch.float32 if shape.io == AS_F32 else torch.bfloat16
        g["dx"] = torch.empty(shape.batch, shape.seqlen, P, dtype=dt, device=device)
    return g


def make_grads(g: dict) -> as_grads_t:
    return as_grads_t(*[_ptr(g[k]) for k in ("dW_delta", "db_delta", "dW_B", "dW_C", "dA_log", "dx")])


def alloc_workspace(nbytes: int, device) -> torch.Tensor:
    return torch.empty(int(nbytes), dtype=torch.uint8, device=device)


# ------------------------------------------------------------------------------------------ entry points
def as_version() -> int:
    return lib().as_version()


def strerror(code: int) -> str:
    return lib().as_strerror(int(code)).decode()


as_strerror = strerror


def as_workspace_bytes(shape: as_shape_t, tbar: int):
    fwd, grad = C.c_size_t(0), C.c_size_t(0)
    _check(lib().as_workspace_bytes(C.byref(shape), int(tbar), C.byref(fwd), C.byref(grad)), "as_workspace_bytes")
    return fwd.value, grad.value


def as_check_status(ws, stream=None) -> int:
    """Status word of the kernels that used `ws`; ws=None reads the built-in scratch of as_ssm_forward_static."""
    return lib().as_check_status(_ptr(ws), _stream(stream))


def as_sm_count() -> int:
    return int(lib().as_sm_count())


def as_ssm_forward(shape, theta, x, y, ws, stream=None):
    p = make_params(theta)
    _check(lib().as_ssm_forward(C.byref(shape), C.byref(p), _ptr(x), _ptr(y), _ptr(ws), ws.numel(), _stream(stream)),
           "as_ssm_forward")


def as_adjoint_grad(shape, theta, x, dy, tbar, grads, ws, flags=0, stream=None):
    p, g = make_params(theta), make_grads(grads)
    _check(lib().as_adjoint_grad(C.byref(shape), C.byref(p), _ptr(x), _ptr(dy), int(tbar), int(flags), C.byref(g),
                                 _ptr(ws), ws.numel(), _stream(stream)), "as_adjoint_grad")


def as_workspace_bytes_layers(shape: as_shape_t, layers: int, tbar: int) -> int:
    grad = C.c_size_t(0)
    _check(lib().as_workspace_bytes_layers(C.byref(shape), int(layers), int(tbar), C.byref(grad)),
           "as_workspace_bytes_layers")
    return grad.value


def as_adjoint_grad_layers(shape, layers, theta, x, dy, tbar, grads, ws, flags=0, stream=None):
    """All layers of a stack in one call: every tensor of `theta` and `grads` has a leading [layers] dimension,
    x is [layers, B, T, P], dy [B, T, P] is shared."""
    p, g = make_params(theta), make_grads(grads)
    _check(lib().as_adjoint_grad_layers(C.byref(shape), int(layers), C.byref(p), _ptr(x), _ptr(dy), int(tbar), int(flags),
                                        C.byref(g), _ptr(ws), ws.numel(), _stream(stream)), "as_adjoint_grad_layers")


def as_wcat_bytes(shape: as_shape_t, layers: int = 1) -> int:
    return int(lib().as_wcat_bytes(C.byref(shape), int(layers)))


def as_pack_weights(shape, layers, theta, wcat, stream=None):
    p = make_params(theta)
    _check(lib().as_pack_weights(C.byref(shape), int(layers), C.byref(p), _ptr(wcat), _stream(stream)), "as_pack_weights")


def alloc_grads_layers(shape: as_shape_t, layers: int, device, with_dx=False) -> dict:
    """Gradient buffers with a leading [layers] dimension for as_adjoint_grad_layers."""
    P, N, K = shape.d_model, shape.d_state, int(layers)
    f = dict(dtype=torch.float32, device=device)
    g = {"dW_delta": torch.empty(K, P, P, **f), "db_delta": torch.empty(K, P, **f), "dW_B": torch.empty(K, N, P, **f),
         "dW_C": torch.empty(K, N, P, **f),
         "dA_log": torch.empty(K, P, **f) if shape.a_structure != AS_A_DIAGONAL else torch.empty(K, P, N, **f), "dx": None}
    if with_dx:
        dt = torch.float32 if shape.io == AS_F32 else torch.bfloat16
        g["dx"] = torch.empty(K, shape.batch, shape.seqlen, P, dtype=dt, device=device)
    return g


def as_full_bptt_grad(shape, theta, x, dy, grads, ws, flags=0, stream=None):
    p, g = make_params(theta), make_grads(grads)
    _check(lib().as_full_bptt_grad(C.byref(shape), C.byref(p), _ptr(x), _ptr(dy), int(flags), C.byref(g),
                                   _ptr(ws), ws.numel(), _stream(stream)), "as_full_bptt_grad")


def as_rmsnorm_fwd(shape, y, yhat, eps=1e-6, stream=None):
    _check(lib().as_rmsnorm_fwd(C.byref(shape), _ptr(y), _ptr(yhat), float(eps), _stream(stream)), "as_rmsnorm_fwd")


def as_residual_add(shape, y_in, ytilde, y_out, stream=None):
    _check(lib().as_residual_add(C.byref(shape), _ptr(y_in), _ptr(ytilde), _ptr(y_out), _stream(stream)),
           "as_residual_add")


def as_rmsnorm_bwd_add(shape, y, dyhat, G_inout, eps=1e-6, stream=None):
    _check(lib().as_rmsnorm_bwd_add(C.byref(shape), _ptr(y), _ptr(dyhat), _ptr(G_inout), float(eps), _stream(stream)),
           "as_rmsnorm_bwd_add")


def as_launch_count(reset: bool = False) -> int:
    return int(lib().as_launch_count(1 if reset else 0))


def as_set_timing(enable: bool):
    _check(lib().as_set_timing(1 if enable else 0), "as_set_timing")


def as_get_timing() -> dict:
    """Milliseconds per phase of the most recent as_adjoint_grad call (timing mode must be on)."""
    ms = (C.c_float * AS_NUM_PHASES)()
    _check(lib().as_get_timing(ms, AS_NUM_PHASES), "as_get_timing")
    return dict(zip(PHASES, [float(v) for v in ms]))


def as_ssm_forward_static(shape, theta, x, y, stream=None):
    """Forward using the library's built-in scratch array: for callers that may not allocate device memory
    (guests of a host program that owns all of it).  Shapes needing more than AS_STATIC_SCRATCH_BYTES of scratch
    raise AsError(AS_ERR_LIMIT).  Calls on one device share the array: do not let two of them overlap."""
    p = make_params(theta)
    _check(lib().as_ssm_forward_static(C.byref(shape), C.byref(p), _ptr(x), _ptr(y), _stream(stream)),
           "as_ssm_forward_static")


def as_wait_selftest(ws, poll_limit=4096, stream=None):
    """Enqueue the bounded-wait self test; afterwards as_check_status(ws) must return AS_ERR_TIMEOUT."""
    _check(lib().as_wait_selftest(_ptr(ws), ws.numel(), int(poll_limit), _stream(stream)), "as_wait_selftest")
