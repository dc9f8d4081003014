#!/usr/bin/env python
"""Benchmark: adjoint-gradient tokens/s per SSM layer at T=65,536, Tbar=2,048 (workload C3).

One "step" = one as_adjoint_grad call (projections, segment pre-pass, carries, main adjoint kernel,
weight-gradient and input-gradient contractions) on one synthetic batch.  Prints ONE JSON line.
`--impl reference` times the fp64 CPU oracle (a deliberately plain program) on a bounded sample.
With --gpus N > 1 (under torchrun) every rank runs an independent replica: the path has no
cross-GPU exchange.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "adjoint-gradient tokens/sec per SSM layer (T=64K, Tbar=2K)"
UNIT = "tokens/s"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks / throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.th = threading.Thread(target=self._read, daemon=True)
            self.th.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
                for n, v in zip(names, r[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            except (ValueError, IndexError):
                continue
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm), "sm_mhz_min": min(sm) if sm else None}


def max_over_ranks(values, device, world):
    """Element-wise maximum over all ranks of a short list of floats (every rank gets the result)."""
    if world <= 1:
        return list(values)
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def job_value(tokens_per_rank, world, ms):
    """Whole-job tokens/s: every rank processed `tokens_per_rank` in the (max-over-ranks) time `ms`."""
    return world * tokens_per_rank / (ms * 1e-3)


def oracle_sample_tokens_per_s(w, sample_T, verbose=False):
    """Time the fp64 oracle (as it stands) on a bounded sample: batch element 0, first sample_T tokens."""
    import numpy as np
    import torch
    from oracle import ssm_oracle as O
    from paper_2501_00692_b200 import synth
    ws = synth.custom_workload(w.name + "-sample", w.config, 1, sample_T, w.d_model, w.d_state, 1,
                               min(w.tbar, sample_T), w.io)
    theta = {k: synth.to_f64(v) for k, v in synth.layer_params(ws, 0, "cpu").items()}
    x, dy = synth.activations(ws, "cpu")
    x, dy = synth.to_f64(x), synth.to_f64(dy)
    c0 = time.process_time()
    t0 = time.perf_counter()
    O.batched(O.adjoint_grad, theta, x, dy, ws.tbar, tier="block")
    dt = time.perf_counter() - t0
    cpu = time.process_time() - c0
    return sample_T / dt, dt, cpu


def cpu_baseline_record(w, sample_T, tps, dt, cpu):
    """What the oracle run really used: the scans are single-threaded numpy loops over time, only the dense products
    (projections, weight and input gradients) run on the BLAS thread pool; `cores` is CPU time / wall time."""
    host = len(os.sched_getaffinity(0))
    return {"value": tps, "unit": UNIT, "cores": max(1, round(cpu / dt)), "kind": "oracle",
            "host_cores": host, "cpu_seconds": round(cpu, 2), "wall_seconds": round(dt, 2),
            "threads": f"1 for the scans (numpy loops over time) + a BLAS pool of up to {host} for the dense products",
            "sample": f"batch element 0, first {sample_T} tokens of {w.name}, Tbar={min(w.tbar, sample_T)}, all "
                      f"{w.d_model} channels ({dt:.1f} s); the whole workload ({w.batch} x {w.seqlen} tokens) would take "
                      f"about {w.batch * w.seqlen / tps:.0f} s, beyond the 10-30 s this leg is allowed"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2501_00692_b200 import synth
    w = synth.WORKLOADS[args.workload]
    sample_T = args.cpu_sample_tokens
    vals = []
    for i in range(args.warmup + args.steps):
        tps, dt, cpu = oracle_sample_tokens_per_s(w, sample_T)
        if i >= args.warmup:
            vals.append((tps, dt, cpu))
    tps = sum(v[0] for v in vals) / len(vals)
    ms = 1e3 * sum(v[1] for v in vals) / len(vals)
    base = cpu_baseline_record(w, sample_T, tps, ms * 1e-3, sum(v[2] for v in vals) / len(vals))
    line = {"impl": "reference", "metric": METRIC, "value": tps, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "batch": 1, "seq_len": sample_T, "d_model": w.d_model,
                       "d_state": w.d_state, "tbar": min(w.tbar, sample_T)},
            "cpu_baseline": base,
            "e2e": {"value": tps, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="C3")
    ap.add_argument("--cpu-sample-tokens", type=int, default=32768)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--batch", type=int, default=None, help="override the workload's batch (profiling runs)")
    ap.add_argument("--seq-len", type=int, default=None, help="override the workload's seqlen (profiling runs)")
    ap.add_argument("--tbar", type=int, default=None, help="override the workload's window (profiling runs)")
    ap.add_argument("--slow-decay", action="store_true", help="slow-decay parameter law (window term live)")
    ap.add_argument("--scalar-a", action="store_true", help="scalar structure: one decay rate per channel (not the headline workload)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)
    if args.impl == "reference":
        args.warmup = min(args.warmup, 1); args.steps = min(args.steps, 3)
        return run_reference(args)
    args.warmup = max(args.warmup, 3)

    import torch
    import torch.distributed as dist
    from paper_2501_00692_b200 import binding as B
    from paper_2501_00692_b200 import synth

    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    B.lib()   # raises if the CUDA library is missing: there is no fallback

    def barrier():
        if world > 1:
            dist.barrier()

    w = synth.WORKLOADS[args.workload]
    if args.batch or args.seq_len or args.tbar:
        w = synth.custom_workload(w.name + "-custom", w.config, args.batch or w.batch, args.seq_len or w.seqlen,
                                  w.d_model, w.d_state, 1, args.tbar or w.tbar, w.io)
    theta = synth.layer_params(w, 0, dev, slow_decay=args.slow_decay)
    x, dy = synth.activations(w, dev)
    if args.scalar_a:
        theta = dict(theta)
        theta["A_log"] = theta["A_log"][:, 0].contiguous()
    sh = B.shape_of(x, w.d_state, a_scalar=args.scalar_a)
    _, gbytes = B.as_workspace_bytes(sh, w.tbar)
    ws = B.alloc_workspace(gbytes, dev)
    grads = B.alloc_grads(sh, dev)
    tokens = w.batch * w.seqlen

    def step(xb=None, dyb=None):
        B.as_adjoint_grad(sh, theta, x if xb is None else xb, dy if dyb is None else dyb, w.tbar, grads, ws)

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()        # samples SM clocks / throttle reasons from here to the end of the timed regions
    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    assert B.as_check_status(ws) == 0
    # ---- device-resident timing --------------------------------------------------------------
    B.as_launch_count(reset=True)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier(); torch.cuda.synchronize()
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    torch.cuda.synchronize(); barrier()
    launches = B.as_launch_count()
    ms = e0.elapsed_time(e1) / args.steps
    # ---- per-phase timing (library-side CUDA events on the launching stream) ---------------------
    B.as_set_timing(True)
    samples = {k: [] for k in B.PHASES}
    for _ in range(max(args.steps, 5)):
        step()
        for k, v in B.as_get_timing().items():
            samples[k].append(v)
    B.as_set_timing(False)
    phase = {k: statistics.median(v) for k, v in samples.items()}   # median over the steps: one slow call moves nothing
    # ---- end to end: pinned host inputs -> device, gradients -> host, inside the timed region -----
    if args.no_e2e:
        ms_e2e, h2d, d2h = float("nan"), 0, 0
    else:
        ms_e2e, h2d, d2h = run_e2e(args, torch, x, dy, grads, step, barrier, e0, e1)

    clocks = sampler.stop() if rank == 0 else None
    ms, ms_e2e = max_over_ranks([ms, ms_e2e if ms_e2e == ms_e2e else -1.0], dev, world)
    if ms_e2e < 0:
        ms_e2e = float("nan")
    report(args, B, w, world, rank, tokens, ms, ms_e2e, h2d, d2h, launches, phase, clocks)
    if world > 1:
        dist.destroy_process_group()


def run_e2e(args, torch, x, dy, grads, step, barrier, e0, e1):
    """End to end with host buffers: every step copies its inputs from pinned host memory to the device and every
    result (the five parameter gradients and dx) back.  The input copies run on a second stream into one of two
    device buffer sets, so step i+1's host->device transfer overlaps step i's kernels, and the dx read-back runs on a
    third stream from a device copy the next step does not overwrite (PCIe, not the kernels, bounds this figure)."""
    xh, dyh = x.cpu().pin_memory(), dy.cpu().pin_memory()
    outh = {k: torch.empty_like(v, device="cpu").pin_memory() for k, v in grads.items() if v is not None}
    h2d = xh.numel() * xh.element_size() * 2
    d2h = sum(v.numel() * v.element_size() for v in outh.values())
    bufs = [(x, dy), (torch.empty_like(x), torch.empty_like(dy))]
    copy_stream, back_stream = torch.cuda.Stream(), torch.cuda.Stream()
    main = torch.cuda.current_stream()
    copied = [torch.cuda.Event() for _ in range(2)]
    consumed = [torch.cuda.Event() for _ in range(2)]
    produced, drained = torch.cuda.Event(), torch.cuda.Event()

    def run(n):
        for i in range(n):
            xb, dyb = bufs[i % 2]
            with torch.cuda.stream(copy_stream):
                if i >= 2:
                    copy_stream.wait_event(consumed[i % 2])      # the kernels of step i-2 are done with this set
                xb.copy_(xh, non_blocking=True); dyb.copy_(dyh, non_blocking=True)
                copied[i % 2].record(copy_stream)
            main.wait_event(copied[i % 2])
            if i >= 1:
                main.wait_event(drained)                         # the previous step's results have left the device buffers
            step(xb, dyb)
            consumed[i % 2].record(main)
            produced.record(main)
            with torch.cuda.stream(back_stream):
                back_stream.wait_event(produced)
                for k, v in outh.items():
                    v.copy_(grads[k], non_blocking=True)
                drained.record(back_stream)
        main.wait_stream(back_stream)

    run(2); torch.cuda.synchronize()
    barrier(); torch.cuda.synchronize()
    e0.record()
    run(args.steps)
    e1.record()
    torch.cuda.synchronize(); barrier()
    return e0.elapsed_time(e1) / args.steps, h2d, d2h


def l2_note(w, tokens):
    """Timing hygiene: what a step streams (x, dy in the I/O dtype, Delta in fp32) against the 126 MB L2."""
    e = 2 if w.io == "bf16" else 4
    gb = tokens * w.d_model * (2 * e + 4) / 1e9
    if gb * 1e9 > 2 * 126e6:
        return f"inputs exceed L2 (x, dy, Delta: {gb:.1f} GB per step), no flush needed"
    return f"inputs fit in L2 ({gb * 1e3:.0f} MB per step): parity workload, not a roofline measurement"


# Per state-step (token, channel, state) work of the main adjoint kernel.
# The method's own count: 1 ex2 (abar_i) + 1 more where the window-exit factor is live, and 12 FP32-pipe operations
# (rebuild h: 3; mu: 2; dC, dB, s: 3; abar h mu and its two sums: 4).  What this build's kernel executes on top of that is
# stated separately, so that redundancy shows instead of being credited.
METHOD_EX2_PER_STATE_STEP = 1.0
METHOD_FMA_PER_STATE_STEP = 12.0
KERNEL_EX2_PER_STATE_STEP = {"forward rebuild of the chunk (abar)": 1.0, "backward walk (abar again)": 1.0,
                             "chunk-start fix-up": 1.0 / 8}
# measured pipe rates per clock per SM (profiles/pipe_rates_microbenchmark.md)
MUFU_PER_CLK_SM = 16.0
FMA_PER_CLK_SM = 128.0


def report(args, B, w, world, rank, tokens, ms, ms_e2e, h2d, d2h, launches, phase, clocks):
    if rank == 0:
        peak, peak_src = measured_peaks()
        e = 2 if w.io == "bf16" else 4
        P, N = w.d_model, w.d_state
        # algorithmic bytes of the main adjoint kernel per token: read x, dy (2 P e), Delta (4 P), B_t, C_t (2 N e);
        # write du, dx_dir (2 P e) and dB_t, dC_t (2 N fp32)
        bytes_per_token = P * (4 * e + 4) + 2 * N * e + 2 * N * 4
        k_ms = phase["adjoint_main"]
        achieved = bytes_per_token * tokens / (k_ms * 1e-3) / 1e9 if k_ms > 0 else None
        sm_mhz = (clocks or {}).get("sm_mhz") or 1965.0
        sms = B.as_sm_count()
        steps = tokens * P * N
        ex2_steps = tokens * P if args.scalar_a else steps    # scalar structure: one decay factor per (token, channel)
        live = 1.0 if args.slow_decay else 0.0            # the window-exit factor is live under the slow-decay law only
        ex2_method = ex2_steps * (METHOD_EX2_PER_STATE_STEP + live)
        fma_method = steps * METHOD_FMA_PER_STATE_STEP
        ex2_exec = ex2_steps * (sum(KERNEL_EX2_PER_STATE_STEP.values()) + live) + tokens * P  # + sigmoid per (token, channel)
        mufu_peak = MUFU_PER_CLK_SM * sms * sm_mhz * 1e6
        fma_peak = FMA_PER_CLK_SM * sms * sm_mhz * 1e6
        sec = k_ms * 1e-3
        alu = {"kernel": "adjoint_main_kernel", "bound": "alu", "sm_mhz": sm_mhz, "launch_ms": k_ms,
               "peak_source": f"{MUFU_PER_CLK_SM:g} ex2 and {FMA_PER_CLK_SM:g} FP32 FMA lanes per clock per SM (measured, "
                              f"profiles/pipe_rates_microbenchmark.md) x {sms} SMs x sampled SM clock",
               "method_ops": {"ex2_per_state_step": METHOD_EX2_PER_STATE_STEP + live, "fma_per_state_step": METHOD_FMA_PER_STATE_STEP},
               "mufu": {"achieved": ex2_method / sec, "peak": mufu_peak, "unit": "ex2/s", "frac": ex2_method / sec / mufu_peak},
               "fma": {"achieved": fma_method / sec, "peak": fma_peak, "unit": "FP32 op/s", "frac": fma_method / sec / fma_peak},
               "executed_ex2": {"per_state_step": KERNEL_EX2_PER_STATE_STEP, "per_launch": ex2_exec,
                                "frac_of_mufu_peak": ex2_exec / sec / mufu_peak}} if k_ms > 0 else None
        traffic = None
        tpath = os.path.join(ROOT, "profiles", "traffic.json")
        if os.path.exists(tpath):
            traffic = json.load(open(tpath)).get(f"adjoint_main_kernel:{w.name}")
        psum = sum(phase.values())
        line = {"metric": METRIC, "value": job_value(tokens, world, ms), "unit": UNIT, "n_gpus": world,
                "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None,
                "dtype": "f32" if w.io == "f32" else "bf16 (fp32 accum)", "data": "synthetic",
                "config": {"workload": w.name, "batch": w.batch, "seq_len": w.seqlen, "d_model": w.d_model,
                           "d_state": w.d_state, "tbar": w.tbar, "io": w.io, "layers": 1,
                           "parallelism": "replicas only" if world > 1 else "single GPU",
                           "l2": l2_note(w, tokens)},
                "e2e": {"value": job_value(tokens, world, ms_e2e) if ms_e2e == ms_e2e else None, "unit": UNIT, "h2d_bytes_per_step": h2d,
                        "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e if ms_e2e == ms_e2e else None,
                        "results_copied_back": "dW_delta, db_delta, dW_B, dW_C, dA_log, dx"},
                "gpu_launches": launches,
                "phases_ms": phase, "phases_sum_ms": psum, "phases_stat": "median over the steps",
                "phases_consistent": abs(psum - ms) <= 0.05 * ms,
                # the metric's named roofline: algorithmic HBM bytes of the dominant kernel / its launch time (library-side
                # CUDA events on the launching stream) against the measured copy bandwidth
                "roofline": {"kernel": "adjoint_main_kernel", "bound": "hbm", "achieved": achieved, "peak": peak,
                             "unit": "GB/s", "frac": (achieved / peak) if achieved else None, "traffic": traffic,
                             "peak_source": peak_src, "bytes_per_token": bytes_per_token,
                             "bytes_per_launch": bytes_per_token * tokens, "launch_ms": k_ms},
                # what actually binds the kernel: MUFU / FP32 issue, on the method's own operation count
                "roofline_alu": alu,
                "clocks": clocks}
        if world == 1 and not args.no_cpu_baseline:
            tps, dt, cpu = oracle_sample_tokens_per_s(w, args.cpu_sample_tokens)
            line["cpu_baseline"] = cpu_baseline_record(w, args.cpu_sample_tokens, tps, dt, cpu)
        print(json.dumps(line))


if __name__ == "__main__":
    main()
