"""Host-only checks of the C-ABI library: it loads, exports every declared symbol, and rejects bad
arguments before launching anything (no GPU needed: every call here fails its argument check)."""
import ctypes as C
import os
import re

import pytest

from paper_2501_00692_b200 import binding as B
from paper_2501_00692_b200.build import build_library

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    build_library()
    return B.lib()


def test_exports_match_header(L):
    hdr = open(os.path.join(ROOT, "include", "adjoint_ssm.h")).read()
    declared = set(re.findall(r"\b(as_[a-z_]+)\s*\(", hdr))
    declared -= {"as_shape_t", "as_params_t", "as_grads_t", "as_dtype_t"}
    assert declared, "no declarations found"
    for name in declared:
        assert hasattr(L, name), f"{name} declared in the header but not exported"
    assert set(B.EXPORTS) == declared
    for name in declared:
        assert name in B.EXPORTS or hasattr(B, name), f"{name} has no Python binding"


def test_version_and_strerror(L):
    assert B.as_version() == 104
    assert B.strerror(0) == "ok"
    assert "tbar" in B.strerror(B.AS_ERR_TBAR)
    assert "unknown" in B.strerror(-999)


def test_struct_layout_matches_c():
    # int32, (pad), int64, 4 x int32  ->  32 bytes with natural alignment
    assert C.sizeof(B.as_shape_t) == 32
    assert B.as_shape_t.seqlen.offset == 8 and B.as_shape_t.d_model.offset == 16 and B.as_shape_t.a_structure.offset == 28
    assert C.sizeof(B.as_params_t) == 48 and C.sizeof(B.as_grads_t) == 48


def test_workspace_query_and_argument_errors(L):
    sh = B.make_shape(2, 65536, 768, 16, B.AS_BF16)
    fwd, grad = B.as_workspace_bytes(sh, 2048)
    assert 0 < fwd < grad < 8 << 30
    for bad, code in ((B.make_shape(0, 8, 64), B.AS_ERR_SHAPE), (B.make_shape(1, 8, 64, 8), B.AS_ERR_SHAPE),
                      (B.make_shape(1, 8, 64, 16, 7), B.AS_ERR_DTYPE), (B.make_shape(1, 8, 60), B.AS_ERR_ALIGN),
                      (B.make_shape(1, 8, 64, 16, B.AS_F32, 5), B.AS_ERR_SHAPE)):
        with pytest.raises(B.AsError) as ei:
            B.as_workspace_bytes(bad, 4)
        assert ei.value.code == code
    with pytest.raises(B.AsError) as ei:
        B.as_workspace_bytes(sh, 0)
    assert ei.value.code == B.AS_ERR_TBAR
    # sizes beyond the 32-bit token-row coordinates or the segment grid dimension are refused, not mis-addressed
    for bad in (B.make_shape(4, 1 << 29, 64), B.make_shape(1, (1 << 31) - 64, 8), B.make_shape(1, 65536 * 2048, 8)):
        with pytest.raises(B.AsError) as ei:
            B.as_workspace_bytes(bad, 4)
        assert ei.value.code == B.AS_ERR_LIMIT
    assert B.as_sm_count() >= 1
    # NULL pointers are rejected before any CUDA call
    p = B.as_params_t(None, None, None, None, None)
    g = B.as_grads_t(None, None, None, None, None, None)
    rc = L.as_adjoint_grad(C.byref(sh), C.byref(p), None, None, 4, 0, C.byref(g), None, 0, None)
    assert rc == B.AS_ERR_NULL
    rc = L.as_ssm_forward(C.byref(sh), C.byref(p), None, None, None, 0, None)
    assert rc == B.AS_ERR_NULL
    # misaligned and undersized workspace (fake, never dereferenced: checks come first)
    ok = C.c_void_p(0x1000)
    p = B.as_params_t(ok, ok, ok, ok, ok)
    g = B.as_grads_t(ok, ok, ok, ok, ok, None)
    assert L.as_adjoint_grad(C.byref(sh), C.byref(p), ok, C.c_void_p(0x1004), 4, 0, C.byref(g), ok, 1 << 40, None) == B.AS_ERR_ALIGN
    assert L.as_adjoint_grad(C.byref(sh), C.byref(p), ok, ok, 4, 0, C.byref(g), ok, 1024, None) == B.AS_ERR_WORKSPACE
    assert L.as_adjoint_grad(C.byref(sh), C.byref(p), ok, ok, 0, 0, C.byref(g), ok, 1 << 40, None) == B.AS_ERR_TBAR
    assert L.as_full_bptt_grad(C.byref(sh), C.byref(p), ok, ok, 0, C.byref(g), ok, 1024, None) == B.AS_ERR_WORKSPACE
    assert L.as_rmsnorm_fwd(C.byref(sh), None, ok, 1e-6, None) == B.AS_ERR_NULL
    # the layers call: same checks, plus the layer count and the limits on layers * batch
    one = B.as_workspace_bytes(sh, 2048)[1]
    many = B.as_workspace_bytes_layers(sh, 4, 2048)
    assert B.as_workspace_bytes_layers(sh, 1, 2048) == one and 3 * one < many < 5 * one
    assert L.as_adjoint_grad_layers(C.byref(sh), 0, C.byref(p), ok, ok, 4, 0, C.byref(g), ok, 1 << 40, None) == B.AS_ERR_SHAPE
    assert L.as_adjoint_grad_layers(C.byref(sh), 3, C.byref(p), ok, ok, 4, 0, C.byref(g), ok, 1024, None) == B.AS_ERR_WORKSPACE
    assert L.as_adjoint_grad_layers(C.byref(sh), 3, C.byref(p), None, ok, 4, 0, C.byref(g), ok, 1 << 40, None) == B.AS_ERR_NULL
    for layers, shape in ((40000, B.make_shape(2, 64, 64)), (1 << 14, B.make_shape(1, 1 << 18, 8))):
        with pytest.raises(B.AsError) as ei:
            B.as_workspace_bytes_layers(shape, layers, 4)
        assert ei.value.code == B.AS_ERR_LIMIT
    # packed weights: size query and argument checks
    assert B.as_wcat_bytes(sh, 3) == 3 * (768 + 32) * 768 * 2 and B.as_wcat_bytes(B.make_shape(0, 8, 64), 1) == 0
    assert L.as_pack_weights(C.byref(sh), 1, C.byref(p), None, None) == B.AS_ERR_NULL
    assert L.as_pack_weights(C.byref(sh), 0, C.byref(p), ok, None) == B.AS_ERR_SHAPE
    f32 = B.make_shape(2, 64, 64)
    assert L.as_pack_weights(C.byref(f32), 1, C.byref(p), ok, None) == B.AS_ERR_DTYPE
    pw = B.as_params_t(ok, ok, ok, ok, ok, C.c_void_p(0x1008))
    assert L.as_adjoint_grad(C.byref(sh), C.byref(pw), ok, ok, 4, 0, C.byref(g), ok, 1 << 40, None) == B.AS_ERR_ALIGN


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", "/nonexistent/libadjoint_ssm.so")
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        B.lib()
