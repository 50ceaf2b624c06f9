#!/usr/bin/env python
"""Benchmark of the block-circulant forward pass: one JSON line per run.

    python bench.py --gpus N --steps K --warmup W            # the CUDA library (C ABI)
    python bench.py --impl reference --steps K --warmup W    # the fp64 dense CPU oracle

A step is one forward pass of the headline workload -- the 4096 x 4096, k = 64, float32 layer with
fused bias + ReLU at batch 256 -- over one batch of seeded synthetic input.  Steps rotate through
enough distinct (layer, x, y) sets that the working set exceeds twice the L2 cache, so every byte
of every step comes from HBM.  With N > 1 (torchrun) every rank runs the same job on its own GPU
and its own batches (samples are independent: no collective on the data path); the reported value
is all samples of all ranks divided by the slowest rank's device time.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import subprocess
import sys
import tempfile
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

from paper_1708_08917_b200 import synth  # noqa: E402

METRIC = "block-circ layer samples/s"
UNIT = "samples/s"
L2_BYTES = 126 * 1024 * 1024

# DRAM traffic of the dominant kernel from one ncu capture (dram__bytes_read.sum + dram__bytes_write.sum
# per launch), valid only while the kernel source is unchanged: the hash ties the counters to the code.
NCU_TRAFFIC = {
    "kernel": None,
    "bytes_per_launch": None,
    "source": "paper_1708_08917_b200/csrc/circ_contract_fma.cu",
    "source_sha256": None,
}


def workload(name: str):
    """The named benchmark workload -> (FcCase, description)."""
    if name.startswith("cfg2_b"):
        b = int(name[len("cfg2_b"):])
        return synth.config2(b), f"FC 4096x4096 k=64 fp32 batch {b}, bias+ReLU fused"
    raise SystemExit(f"unknown workload {name}")


def algorithmic_bytes(case, sx=4, sy=4, sw=4) -> int:
    """Bytes the method itself must move per forward: stored spectra + x + y + bias."""
    return sw * case.m * case.n // case.k + sx * case.batch * case.n + sy * case.batch * case.m + (4 * case.m if case.bias is not None else 0)


def measured_peaks() -> dict:
    f = ROOT / "MEASURED_PEAKS.json"
    if f.exists():
        d = json.loads(f.read_text())
        return {"hbm_gbs": float(d["hbm_gbs"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "source": "fallback"}


class ClockSampler:
    """nvidia-smi clock / throttle samples taken while the timed region runs (read-only queries)."""
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        self.index = device_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.index)], stdout=self.tmp, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is not None:
            self.proc.terminate()          # the exact child we started
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        self.tmp.flush()
        self.tmp.seek(0)
        sm, smax, reasons = [], [], set()
        for line in self.tmp.read().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                smax.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.tmp.close()
        os.unlink(self.tmp.name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def oracle_rate(case, budget_s: float = 12.0):
    """Time the fp64 dense oracle, as it stands, on a bounded number of batch rows -> (samples/s, rows, threads, seconds)."""
    import oracle
    w = case.w.astype(np.float64)
    x = case.x.astype(np.float64)
    bias = None if case.bias is None else case.bias.astype(np.float64)
    t0 = time.perf_counter()
    oracle.fc(w, x[:1], bias=bias, relu=case.relu)
    per_row = max(time.perf_counter() - t0, 1e-6)
    rows = int(min(case.batch, max(oracle.threads(), budget_s * oracle.threads() / per_row / 4)))
    rows = max(1, min(rows, case.batch))
    t0 = time.perf_counter()
    oracle.fc(w, x[:rows], bias=bias, relu=case.relu)
    dt = time.perf_counter() - t0
    return rows / dt, rows, oracle.threads(), dt


def run_reference(args) -> int:
    """The reference arm: the CPU oracle on the same config / metric; rank 0 only."""
    if int(os.environ.get("RANK", "0")) != 0:
        return 0
    case, desc = workload(args.workload)
    import oracle
    w = case.w.astype(np.float64)
    bias = None if case.bias is None else case.bias.astype(np.float64)
    x = case.x.astype(np.float64)
    # bounded sample of the batch per step, sized so that the whole run stays within about two minutes
    t0 = time.perf_counter()
    oracle.fc(w, x[:1], bias=bias, relu=case.relu)
    t_row = max(time.perf_counter() - t0, 1e-6)
    rows = int(max(1, min(case.batch, 120.0 / ((args.steps + args.warmup) * t_row))))
    for _ in range(args.warmup):
        oracle.fc(w, x[:rows], bias=bias, relu=case.relu)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.fc(w, x[:rows], bias=bias, relu=case.relu)
    dt = time.perf_counter() - t0
    value = rows * args.steps / dt
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "description": desc, "sample": f"{rows} of {case.batch} batch rows per step"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
                         "sample": f"{rows} of {case.batch} batch rows per step, all outputs"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


def max_over_ranks(ms: float, world: int) -> float:
    """Slowest rank's device time (all-reduce MAX over the process group when there is one)."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device="cuda" if dist.get_backend() == "nccl" else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def traffic_if_current():
    src = ROOT / NCU_TRAFFIC["source"]
    if NCU_TRAFFIC["bytes_per_launch"] is None or not src.exists():
        return None
    if hashlib.sha256(src.read_bytes()).hexdigest() != NCU_TRAFFIC["source_sha256"]:
        return None        # the kernel changed since the counters were taken
    return NCU_TRAFFIC["bytes_per_launch"]


def run_ours(args) -> int:
    import torch
    import paper_1708_08917_b200 as circ

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    case, desc = workload(args.workload)
    B = case.batch
    alg = algorithmic_bytes(case)
    # distinct (layer, x, y) sets so that consecutive steps never touch the same bytes: > 2 x L2
    per_set = alg + 3 * 4 * case.m * case.n // case.k + 8 * B * (case.m + case.n)   # + embedded operand + workspace
    sets = int(min(64, max(2, -(-2 * L2_BYTES // per_set) + 1)))
    stream = torch.cuda.current_stream()
    handles, xs, ys = [], [], []
    for s in range(sets):
        h = circ.circ_fc_create(case.m, case.n, case.k, case.w)
        if case.bias is not None:
            circ.circ_set_bias(h, case.bias)
        circ.circ_set_activation(h, int(case.relu))
        circ.circ_reserve(h, B)
        handles.append(h)
        # every set and every rank gets its own batch (same distribution, different stream id)
        xs.append(torch.from_numpy(synth.uniform((B, case.n), -1.0, 1.0, synth.stream_id(case.name, f"x{rank}_{s}"))).cuda())
        ys.append(torch.empty(B, case.m, device="cuda", dtype=torch.float32))
    torch.cuda.synchronize()

    def step(i):
        s = i % sets
        circ.circ_fc_forward(handles[s], xs[s], ys[s], B, stream)

    for i in range(max(args.warmup, 3)):
        step(i)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = circ.circ_launch_count()
    torch.cuda.synchronize()
    e0.record(stream)
    for i in range(args.steps):
        step(i)
    e1.record(stream)
    torch.cuda.synchronize()
    launches = circ.circ_launch_count() - launches0
    if world > 1:
        dist.barrier()
    clocks = sampler.stop()
    ms_total = max_over_ranks(e0.elapsed_time(e1), world)
    ms_step = ms_total / args.steps
    value = world * B * args.steps / (ms_total * 1e-3)
    variant = circ.circ_last_variant(handles[0])

    # per-kernel device times over the same rotation (separate pass: events between kernels)
    prof_steps = min(args.steps, 200)
    for h in handles:
        circ.circ_profile_begin(h)
    for i in range(prof_steps):
        step(i)
    torch.cuda.synchronize()
    stage_ms, stage_n = [0.0] * 4, [0] * 4
    for h in handles:
        ms, cnt = circ.circ_profile_end(h)
        stage_ms = [a + b for a, b in zip(stage_ms, ms)]
        stage_n = [a + b for a, b in zip(stage_n, cnt)]
    names = ["input_fft", "contraction", "output_ifft", "fused_fc"]
    per_launch_us = {names[i]: (1e3 * stage_ms[i] / stage_n[i] if stage_n[i] else None) for i in range(4)}
    dom = max(range(4), key=lambda i: stage_ms[i])
    dom_us = 1e3 * stage_ms[dom] / max(stage_n[dom], 1)
    peaks = measured_peaks()
    achieved = alg / (dom_us * 1e-6) / 1e9
    roofline = {"bound": "hbm", "kernel": names[dom], "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"], "peak_source": peaks["source"], "frac_of_nominal_8000": achieved / 8000.0,
                "traffic": traffic_if_current(), "algorithmic_bytes_per_launch": alg,
                "kernel_us_per_launch": per_launch_us,
                "whole_forward_frac": alg / (ms_step * 1e-3) / 1e9 / peaks["hbm_gbs"]}

    # end to end through the host-pointer entry point: pinned host x -> device -> forward -> pinned host y
    e2e = None
    if True:
        xh = [torch.from_numpy(synth.uniform((B, case.n), -1.0, 1.0, synth.stream_id(case.name, f"xh{rank}_{s}"))).pin_memory()
              for s in range(min(sets, 8))]
        yh = [torch.empty(B, case.m, dtype=torch.float32).pin_memory() for _ in range(len(xh))]
        for i in range(3):
            circ.circ_fc_forward_host(handles[i % sets], xh[i % len(xh)], yh[i % len(xh)], B, stream)
        torch.cuda.synchronize()
        e2e_steps = min(args.steps, 300)
        if world > 1:
            dist.barrier()
        e0.record(stream)
        for i in range(e2e_steps):
            circ.circ_fc_forward_host(handles[i % sets], xh[i % len(xh)], yh[i % len(xh)], B, stream)
        e1.record(stream)
        torch.cuda.synchronize()
        ms_e2e = max_over_ranks(e0.elapsed_time(e1), world)
        e2e = {"value": world * B * e2e_steps / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": 4 * B * case.n,
               "d2h_bytes_per_step": 4 * B * case.m, "steps": e2e_steps}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        rate, rows, threads, secs = oracle_rate(case)
        cpu = {"value": rate, "unit": UNIT, "cores": threads, "kind": "oracle",
               "sample": f"{rows} of {B} batch rows, all {case.m} outputs, {secs:.1f} s"}

    for h in handles:
        circ.circ_destroy(h)
    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic",
            "config": {"workload": args.workload, "description": desc, "batch_per_gpu": B, "variant": variant,
                       "l2": f"steps rotate through {sets} distinct (layer, x, y) sets, {sets * per_set / 1e6:.0f} MB > 2 x L2",
                       "dense_equiv_tflops": 2.0 * case.m * case.n * B * world / (ms_step * 1e-3) / 1e12},
            "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": int(launches), "clocks": clocks,
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def main() -> int:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2_b256")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
