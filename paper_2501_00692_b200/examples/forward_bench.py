"""Times `as_ssm_forward` on one workload for the diagonal structure (scan kernels) and the scalar structure (bf16 I/O,
d_model % 128 == 0: y pass in the matmul form), CUDA events, median over the calls.

    python -m paper_2501_00692_b200.examples.forward_bench [--workload C3] [--batch B --seq-len T --d-model P] [--calls 20]
"""
import argparse

import torch

from paper_2501_00692_b200 import binding as B
from paper_2501_00692_b200 import synth


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="C3")
    ap.add_argument("--batch", type=int)
    ap.add_argument("--seq-len", type=int)
    ap.add_argument("--d-model", type=int)
    ap.add_argument("--calls", type=int, default=20)
    ap.add_argument("--only", choices=["diagonal", "scalar"])
    a = ap.parse_args()
    base = synth.WORKLOADS[a.workload]
    w = synth.custom_workload("forward-bench", base.config, a.batch or base.batch, a.seq_len or base.seqlen,
                              a.d_model or base.d_model, io="bf16")
    dev = "cuda:0"
    theta = dict(synth.layer_params(w, 0, dev))
    x, _ = synth.activations(w, dev)
    tied = dict(theta)
    tied["A_log"] = theta["A_log"][:, 5].contiguous()
    for tag, th, kw in (("diagonal", theta, {}), ("scalar", tied, {"a_scalar": True})):
        if a.only and a.only != tag:
            continue
        sh = B.shape_of(x, w.d_state, **kw)
        ws = B.alloc_workspace(B.as_workspace_bytes(sh, w.seqlen)[0], dev)
        y = torch.empty_like(x)
        for _ in range(3):
            B.as_ssm_forward(sh, th, x, y, ws)
        torch.cuda.synchronize()
        ts = []
        for _ in range(a.calls):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            B.as_ssm_forward(sh, th, x, y, ws)
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        ts.sort()
        assert B.as_check_status(ws) == 0
        ms = ts[len(ts) // 2]
        print(f"{tag:10s} as_ssm_forward {ms:.4f} ms  {w.batch * w.seqlen / ms / 1e3:.1f} M tokens/s")

if __name__ == "__main__":
    main()
