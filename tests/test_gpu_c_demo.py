"""The boundary is a C ABI: a plain-C program (no Python, no torch in the process) links the library, feeds it raw
buffers and must produce what the Python binding produces on the same inputs."""
import os
import subprocess

import numpy as np
import pytest
import torch

from paper_2501_00692_b200 import binding as B
from paper_2501_00692_b200 import synth
from paper_2501_00692_b200.build import LIB, build_library

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_plain_c_caller_matches_the_binding(tmp_path):
    build_library()
    src = os.path.join(ROOT, "paper_2501_00692_b200", "examples", "demo_c_abi.c")
    exe = str(tmp_path / "demo_c_abi")
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    libdir = os.path.dirname(LIB)
    subprocess.run([nvcc, "-x", "c", src, "-o", exe, "-L" + libdir, "-ladjoint_ssm", "-lcudart",
                    "-Xlinker", "-rpath=" + libdir], check=True)
    w = synth.custom_workload("cdemo", 27, 2, 900, 72, tbar=130, io="f32")
    theta = synth.layer_params(w, 0, DEV, slow_decay=True)
    x, dy = synth.activations(w, DEV)
    order = [theta[k] for k in ("W_delta", "b_delta", "W_B", "W_C", "A_log")] + [x, dy]
    with open(tmp_path / "in.bin", "wb") as f:
        for t in order:
            f.write(t.detach().float().cpu().numpy().tobytes())
    r = subprocess.run([exe, str(w.batch), str(w.seqlen), str(w.d_model), str(w.tbar), str(tmp_path / "in.bin"),
                        str(tmp_path / "out.bin")], capture_output=True, text=True)
    assert r.returncode == 0, r.stdout + r.stderr
    sh = B.shape_of(x, w.d_state)
    _, gb = B.as_workspace_bytes(sh, w.tbar)
    ws = B.alloc_workspace(gb, DEV)
    g = B.alloc_grads(sh, DEV)
    y = torch.empty_like(x)
    B.as_ssm_forward(sh, theta, x, y, ws)
    B.as_adjoint_grad(sh, theta, x, dy, w.tbar, g, ws)
    torch.cuda.synchronize()
    raw = np.fromfile(tmp_path / "out.bin", dtype=np.float32)
    off = 0
    for name, ref in [("y", y), ("dW_delta", g["dW_delta"]), ("db_delta", g["db_delta"]), ("dW_B", g["dW_B"]),
                      ("dW_C", g["dW_C"]), ("dA_log", g["dA_log"]), ("dx", g["dx"])]:
        n = ref.numel()
        got = raw[off:off + n].reshape(tuple(ref.shape)); off += n
        want = ref.float().cpu().numpy()
        assert np.abs(got - want).max() <= 1e-5 * max(np.abs(want).max(), 1e-30), name
    assert off == raw.size
