#!/usr/bin/env python
"""Benchmark of the block-circulant forward pass: one JSON line per run.

    python bench.py --gpus N --steps K --warmup W            # the CUDA library (C ABI)
    python bench.py --impl reference --steps K --warmup W    # the fp64 dense CPU oracle
    python bench.py --workload NAME ...                      # another configuration (see workload())

A step is one forward pass of the workload over one batch of seeded synthetic input.  The default
workload is the 4096 x 4096, k = 64, float32 layer with fused bias + ReLU at batch 256.  Steps
rotate through enough distinct (layer, x, y) sets that the working set exceeds twice the L2 cache,
so every byte of every step comes from HBM.  With N > 1 (torchrun) every rank runs the same job on
its own GPU and its own batches (samples are independent: no collective on the data path); the
reported value is all samples of all ranks divided by the slowest rank's device time.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import re
import subprocess
import sys
import tempfile
import time
from dataclasses import dataclass
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

from paper_1708_08917_b200 import synth  # noqa: E402

METRIC = "block-circ layer samples/s"
UNIT = "samples/s"
L2_BYTES = 126 * 1024 * 1024
STAGES = ["input_fft", "contraction", "output_ifft", "fused_fc"]
STAGE_SOURCE = {"input_fft": "circ_staged.cu", "output_ifft": "circ_staged.cu", "contraction": "circ_tensor.cu",
                "fused_fc": "circ_fused.cu"}

# DRAM traffic per launch from ncu captures (dram__bytes_read.sum + dram__bytes_write.sum), keyed by
# (workload, kernel).  Each entry is tied to the sha256 of the kernel's source file at capture time;
# when the source has changed since, the figure is withheld (reported as null).
NCU_TRAFFIC: dict = {
    # profiles/dram_traffic_cfg2_b256.md
    ("cfg2_b256", "input_fft"): {"bytes_per_launch": 4211584, "source_sha256": "2c4296cd4a497d41ba9e2d60a62486c6d2ac62b9ec2d83c1bab715597c1b48b4"},
    ("cfg2_b256", "contraction"): {"bytes_per_launch": 6311936, "source_sha256": "498aaea78199b3c537fdee7af01a5671ff0e1fe543c51cc803d19aac3fb85d99"},
    ("cfg2_b256", "output_ifft"): {"bytes_per_launch": 4230400, "source_sha256": "2c4296cd4a497d41ba9e2d60a62486c6d2ac62b9ec2d83c1bab715597c1b48b4"},
    # profiles/fused_fc_kernel_sweep_n16384_k4_b1.md (dram read + write of one launch)
    ("sweep_n16384_k4_b1", "fused_fc"): {"bytes_per_launch": 275349504, "source_sha256": "dbc004fed09f19ed5d3f515d7ea5396d7c2822a051f4ceaeff60c43cd455ddde"},
    # profiles/contract_tc_kernel_sweep_n16384_k4_b1024.md
    ("sweep_n16384_k4_b1024", "contraction"): {"bytes_per_launch": 647336448, "source_sha256": "498aaea78199b3c537fdee7af01a5671ff0e1fe543c51cc803d19aac3fb85d99"},
}


@dataclass
class Workload:
    name: str
    desc: str
    kind: str            # "fc" or "conv"
    case: object
    samples: int         # samples (FC) or images (CONV) per step
    alg_bytes: int       # bytes the method must move per forward
    dense_flops: float   # flops of the equivalent dense layer per forward
    sx: int
    sy: int
    contraction_flops: float = 0.0   # p q B (4k - 4) (x taps): flops of the per-frequency products
    spectra_bf16: bool = False       # the streaming kernel reads bfloat16 weight spectra (workload suffix _w16)


def workload(name: str) -> Workload:
    """Named workloads: cfg1, cfg2_b{B}, cfg3_l{0,1,2}, cfg3_stack, cfg4, sweep_n{n}_k{k}_b{B}[_bf16][_w16]."""
    def fc(case, desc, w16=False):
        s = 2 if case.bf16_io else 4
        alg = (2 if w16 else 4) * case.m * case.n // case.k + s * case.batch * (case.n + case.m) + (4 * case.m if case.bias is not None else 0)
        p, q = case.m // case.k, case.n // case.k
        return Workload(name, desc, "fc", case, case.batch, alg, 2.0 * case.m * case.n * case.batch, s, s,
                        float(p) * q * case.batch * (4 * case.k - 4), w16)

    if name == "cfg1":
        return fc(synth.config1(), "FC 256x256 k=16 fp32 batch 1")
    m = re.fullmatch(r"cfg2_b(\d+)", name)
    if m:
        b = int(m.group(1))
        return fc(synth.config2(b), f"FC 4096x4096 k=64 fp32 batch {b}, bias+ReLU fused")
    m = re.fullmatch(r"cfg3_l([012])", name)
    if m:
        c = synth.config3_layers(128)[int(m.group(1))]
        if c.x.shape[0] != 128:
            c.x = synth.normal((128, c.n), 1.0, synth.stream_id(c.name, "x"), absolute=True)
        return fc(c, f"FC {c.n}->{c.m} k=128 fp32 batch 128 (AlexNet-FC stack layer {m.group(1)})")
    m = re.fullmatch(r"sweep_n(\d+)_k(\d+)_b(\d+)(_bf16)?(_w16)?", name)
    if m:
        n, k, b, bf, w16 = int(m.group(1)), int(m.group(2)), int(m.group(3)), bool(m.group(4)), bool(m.group(5))
        if w16 and b > 8:
            raise SystemExit("_w16 (bfloat16 weight spectra) applies to the small-batch streaming kernel: batch <= 8")
        return fc(synth.sweep_point(n, k, b, bf),
                  f"FC {n}x{n} k={k} {'bf16' if bf else 'fp32'} batch {b}" + (", bf16 weight spectra" if w16 else ""), w16)
    if name == "cfg3_stack":
        layers = synth.config3_layers(128)
        first, last = layers[0], layers[-1]
        # what the stack must move: every layer's defining vectors once, the input and the final output;
        # the activations between the layers need not touch memory
        alg = sum(4 * l.m * l.n // l.k for l in layers) + 4 * 128 * (first.n + last.m)
        stack = synth.FcCase("cfg3_stack", last.m, first.n, first.k, 128, None, first.x, None, False, False)
        stack.layers = layers
        return Workload(name, "FC stack 9216->4096->4096->1024 k=128 fp32 batch 128, ReLU between layers, one circ_stack_forward",
                        "stack", stack, 128, alg, sum(2.0 * l.m * l.n * 128 for l in layers), 4, 4,
                        sum(float(l.m // l.k) * (l.n // l.k) * 128 * (4 * l.k - 4) for l in layers))
    if name == "cfg4":
        c = synth.config4()
        pix = c.N * c.H * c.W
        alg = 4 * c.r * c.r * c.c_out * c.c_in // c.k + 2 * pix * (c.c_in + c.c_out)
        return Workload(name, "CONV 3x3 pad 1, 256->256 ch, 28x28, batch 32, k=16, bf16 activations", "conv", c, c.N, alg,
                        2.0 * pix * c.r * c.r * c.c_in * c.c_out, 2, 2,
                        float(c.r * c.r) * (c.c_out // c.k) * (c.c_in // c.k) * pix * (4 * c.k - 4))
    raise SystemExit(f"unknown workload {name}")


def measured_peaks() -> dict:
    f = ROOT / "MEASURED_PEAKS.json"
    if f.exists():
        d = json.loads(f.read_text())
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1400.0, "source": "fallback"}


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
                                          "-lms", "50", "-i", str(self.index)], stdout=self.tmp, stderr=subprocess.DEVNULL)
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


# ---- the oracle legs (CPU) -----------------------------------------------------------------------

def oracle_forward(wl: Workload, units: int):
    """Run the fp64 dense oracle on the first `units` samples (FC rows / CONV images) of the workload."""
    import oracle
    c = wl.case
    bias = None if c.bias is None else c.bias.astype(np.float64)
    if wl.kind == "stack":
        a = c.x[:units].astype(np.float64)
        for l in c.layers:
            a = oracle.fc(l.w.astype(np.float64), a, relu=l.relu)
        return a
    if wl.kind == "fc":
        return oracle.fc(c.w.astype(np.float64), c.x[:units].astype(np.float64), bias=bias, relu=c.relu)
    return oracle.conv(c.w.astype(np.float64), c.x[:units].astype(np.float64), c.pad, bias=bias, relu=c.relu)


def oracle_rate(wl: Workload, budget_s: float = 12.0):
    """Time the oracle, as it stands, for about `budget_s` seconds on a bounded sample -> (samples/s, description, threads)."""
    import oracle
    t0 = time.perf_counter()
    oracle_forward(wl, 1)
    t_one = max(time.perf_counter() - t0, 1e-6)
    units = int(max(1, min(wl.samples, budget_s / t_one / 2)))
    done, t0 = 0, time.perf_counter()
    while True:
        oracle_forward(wl, units)
        done += units
        dt = time.perf_counter() - t0
        if dt >= budget_s or done >= 50 * wl.samples:
            break
    what = "images" if wl.kind == "conv" else "batch rows"
    return done / dt, f"{units} of {wl.samples} {what} per pass, {done // units} passes, all outputs, {dt:.1f} s", oracle.threads()


def run_reference(args) -> int:
    """The reference arm: the CPU oracle on the same config / metric; rank 0 only."""
    if int(os.environ.get("RANK", "0")) != 0:
        return 0
    wl = workload(args.workload)
    import oracle
    # bounded sample of the batch per step, sized so that the whole run stays within about two minutes
    t0 = time.perf_counter()
    oracle_forward(wl, 1)
    t_one = max(time.perf_counter() - t0, 1e-6)
    units = int(max(1, min(wl.samples, 120.0 / ((args.steps + args.warmup) * t_one))))
    for _ in range(args.warmup):
        oracle_forward(wl, units)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_forward(wl, units)
    dt = time.perf_counter() - t0
    value = units * args.steps / dt
    sample = f"{units} of {wl.samples} {'images' if wl.kind == 'conv' else 'batch rows'} per step, all outputs"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "description": wl.desc, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


# ---- the CUDA arm ----------------------------------------------------------------------------------

def max_over_ranks(ms: float, world: int) -> float:
    """Slowest rank's device time (all-reduce MAX over the process group when there is one)."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device="cuda" if dist.get_backend() == "nccl" else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def traffic_if_current(wl_name: str, kernel: str):
    ent = NCU_TRAFFIC.get((wl_name, kernel))
    if not ent:
        return None
    src = ROOT / "paper_1708_08917_b200" / "csrc" / STAGE_SOURCE[kernel]
    if not src.exists() or hashlib.sha256(src.read_bytes()).hexdigest() != ent["source_sha256"]:
        return None        # the kernel changed since the counters were taken
    return ent["bytes_per_launch"]


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

    wl = workload(args.workload)
    c = wl.case
    tdt = torch.bfloat16 if c.bf16_io else torch.float32
    if wl.kind == "fc":
        x_shape, y_shape = (c.batch, c.n), (c.batch, c.m)
        weight_store = 3 * 4 * c.m * c.n // c.k + 4 * c.m * c.n // c.k      # stream + embedded f32 + embedded bf16 hi/lo
        workspace = 4 * (c.batch + 1) * (c.m + c.n)
    elif wl.kind == "stack":
        x_shape, y_shape = (c.batch, c.n), (c.batch, c.m)
        weight_store = sum(16 * l.m * l.n // l.k for l in c.layers)
        workspace = sum(4 * (c.batch + 1) * (l.m + l.n) for l in c.layers)
    else:
        Ho, Wo = c.H + 2 * c.pad - c.r + 1, c.W + 2 * c.pad - c.r + 1
        x_shape, y_shape = (c.N, c.H, c.W, c.c_in), (c.N, Ho, Wo, c.c_out)
        weight_store = 4 * 4 * c.r * c.r * c.c_out * c.c_in // c.k
        workspace = 4 * (c.N + 1) * c.H * c.W * (c.c_in + c.c_out)
    per_set = wl.alg_bytes + weight_store + workspace
    # distinct (layer, x, y) sets so that consecutive steps never touch the same bytes: > 2 x L2
    sets = int(min(args.max_sets, max(2, -(-2 * L2_BYTES // per_set) + 1)))
    stream = torch.cuda.current_stream()

    def draw_x(tag):
        if wl.kind == "fc":
            a = synth.uniform(x_shape, -1.0, 1.0, synth.stream_id(c.name, tag))
        else:   # CONV and the FC stack take post-ReLU-like activations
            a = synth.normal(x_shape, 1.0, synth.stream_id(c.name, tag), absolute=True)
        return torch.from_numpy(a)

    handles, xs, ys, stacks, stack_layers = [], [], [], [], []
    for s in range(sets):
        if wl.kind == "stack":
            hs = []
            for l in c.layers:
                hl = circ.circ_fc_create(l.m, l.n, l.k, l.w)
                circ.circ_set_activation(hl, int(l.relu))
                if args.variant:
                    circ.circ_set_variant(hl, args.variant)
                hs.append(hl)
            st_h = circ.circ_stack_create(hs)
            circ.circ_stack_reserve(st_h, c.batch)
            stack_layers.append(hs)
            stacks.append(st_h)
            xs.append(draw_x(f"x{rank}_{s}").cuda().to(tdt))
            ys.append(torch.empty(y_shape, device="cuda", dtype=tdt))
            continue
        if wl.kind == "fc":
            h = circ.circ_fc_create(c.m, c.n, c.k, c.w)
            circ.circ_reserve(h, c.batch)
        else:
            h = circ.circ_conv_create(c.c_out, c.c_in, c.r, c.pad, c.k, c.w)
            circ.circ_reserve(h, c.N * c.H * c.W)
        if c.bias is not None:
            circ.circ_set_bias(h, c.bias)
        circ.circ_set_activation(h, int(c.relu))
        code = circ.CIRC_BF16 if c.bf16_io else circ.CIRC_F32
        circ.circ_set_io_dtype(h, code, code)
        if wl.spectra_bf16:
            circ.circ_set_spectrum_dtype(h, circ.CIRC_BF16)
        if args.variant:
            circ.circ_set_variant(h, args.variant)
        handles.append(h)
        # every set and every rank gets its own batch (same distribution, different stream id)
        xs.append(draw_x(f"x{rank}_{s}").cuda().to(tdt))
        ys.append(torch.empty(y_shape, device="cuda", dtype=tdt))
    torch.cuda.synchronize()

    def forward(s, st):
        if wl.kind == "stack":
            circ.circ_stack_forward(stacks[s], xs[s], ys[s], c.batch, st)
        elif wl.kind == "fc":
            circ.circ_fc_forward(handles[s], xs[s], ys[s], c.batch, st)
        else:
            circ.circ_conv_forward(handles[s], xs[s], ys[s], c.N, c.H, c.W, st)

    for i in range(max(args.warmup, 3)):
        forward(i % sets, stream)
    torch.cuda.synchronize()
    circ.circ_device_status(stack_layers[0][0] if wl.kind == "stack" else handles[0])

    # One rotation through all sets is captured in a CUDA graph so that the GPU, not the host's
    # launch rate, sets the pace; the timed region replays it and runs the remainder eagerly.
    graph, cap_stream = torch.cuda.CUDAGraph(), torch.cuda.Stream()
    cap_stream.wait_stream(stream)
    l0 = circ.circ_launch_count()
    with torch.cuda.graph(graph, stream=cap_stream):
        cs = torch.cuda.current_stream()
        if args.streams <= 1:
            for s in range(sets):
                forward(s, cs)
        else:
            # independent batches on `streams` parallel branches of the graph (each set has its own layer,
            # input, output and workspace): throughput of a server that keeps several requests in flight
            branches = [torch.cuda.Stream() for _ in range(args.streams)]
            for b in branches:
                b.wait_stream(cs)
            for s in range(sets):
                forward(s, branches[s % args.streams])
            for b in branches:
                cs.wait_stream(b)
    launches_per_rotation = circ.circ_launch_count() - l0
    graph.replay()
    torch.cuda.synchronize()
    replays, rest = divmod(args.steps, sets)

    if world > 1:
        dist.barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = circ.circ_launch_count()
    torch.cuda.synchronize()
    e0.record(stream)
    for _ in range(replays):
        graph.replay()
    for i in range(rest):
        forward(i % sets, stream)
    e1.record(stream)
    torch.cuda.synchronize()
    launches = circ.circ_launch_count() - launches0 + replays * launches_per_rotation
    if world > 1:
        dist.barrier()
    clocks = sampler.stop()
    ms_total = max_over_ranks(e0.elapsed_time(e1), world)
    ms_step = ms_total / args.steps
    value = world * wl.samples * args.steps / (ms_total * 1e-3)
    variant = circ.circ_last_variant(stack_layers[0][0] if wl.kind == "stack" else handles[0])

    # Per-kernel device times, measured with the same CUDA events on the same rotating buffers: the
    # rotation is captured again with ONE stage's kernel launched 1 + R times per forward (each of
    # these kernels rewrites its own output from unchanged inputs), and the extra time per extra
    # launch is that kernel's duration.  Unlike events around single launches this carries no
    # per-event overhead, which would double the reading for kernels of a few microseconds.
    def time_rotation(nrep, nstreams=1):
        g2, cs2 = torch.cuda.CUDAGraph(), torch.cuda.Stream()
        cs2.wait_stream(stream)
        with torch.cuda.graph(g2, stream=cs2):
            st = torch.cuda.current_stream()
            if nstreams <= 1:
                for s_ in range(sets):
                    forward(s_, st)
            else:
                br = [torch.cuda.Stream() for _ in range(nstreams)]
                for b_ in br:
                    b_.wait_stream(st)
                for s_ in range(sets):
                    forward(s_, br[s_ % nstreams])
                for b_ in br:
                    st.wait_stream(b_)
        g2.replay()
        torch.cuda.synchronize()
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record(stream)
        for _ in range(nrep):
            g2.replay()
        a1.record(stream)
        torch.cuda.synchronize()
        return a0.elapsed_time(a1) / (nrep * sets)       # ms per forward

    R = 3
    nrep = max(3, min(200, args.steps // sets // 4))
    used_stages = [] if wl.kind == "stack" else [3] if variant == circ.CIRC_VARIANT_FUSED else [0, 1, 2]
    base_ms = time_rotation(nrep)
    stage_ms = [0.0] * 4
    for st_i in used_stages:
        for h in handles:
            circ.circ_set_stage_repeat(h, st_i, 1 + R)
        stage_ms[st_i] = max(0.0, (time_rotation(nrep) - base_ms) / R)
        for h in handles:
            circ.circ_set_stage_repeat(h, st_i, 1)
    per_launch_us = {STAGES[i]: (1e3 * stage_ms[i] if i in used_stages else None) for i in range(4)}
    # context only: the same rotation with four independent batches in flight (four graph branches)
    overlap4 = world * wl.samples / (time_rotation(nrep, 4) * 1e-3) if sets >= 4 else None
    peaks = measured_peaks()
    if wl.kind == "stack":
        # seven kernels of three kinds: the roofline is taken over the whole call (every layer's defining vectors,
        # the input and the output once, against the HBM peak); per-kernel figures are those of the cfg3_l* workloads
        dom, dom_us = 2, 1e3 * ms_step
        STAGE_NAME = "whole_stack"
    else:
        dom = max(used_stages, key=lambda i: stage_ms[i])
        dom_us = max(1e3 * stage_ms[dom], 1e-3)
        STAGE_NAME = STAGES[dom]
    # Which roofline bounds the dominant kernel: the contraction is tensor-bound when its flops at the
    # tensor peak (a third of the bf16 peak for float32 inputs: three bf16 passes) take longer than the
    # forward's algorithmic bytes at the HBM peak; everything else is HBM-bound.
    tensor_peak = peaks["bf16_tflops"] / (1.0 if c.bf16_io else 3.0)
    t_hbm = wl.alg_bytes / (peaks["hbm_gbs"] * 1e9)
    t_tc = wl.contraction_flops / (tensor_peak * 1e12)
    if STAGE_NAME == "contraction" and variant == circ.CIRC_VARIANT_TENSOR and t_tc > t_hbm:
        achieved = wl.contraction_flops / (dom_us * 1e-6) / 1e12
        roofline = {"bound": "tensor", "kernel": STAGES[dom], "achieved": achieved, "peak": tensor_peak, "unit": "TFLOP/s",
                    "frac": achieved / tensor_peak, "peak_source": peaks["source"],
                    "peak_note": "measured sustained bf16 GEMM rate" + ("" if c.bf16_io else " / 3 (hi*hi + lo*hi + hi*lo passes)"),
                    "traffic": traffic_if_current(wl.name, STAGES[dom]), "algorithmic_flops_per_launch": wl.contraction_flops}
    else:
        achieved = wl.alg_bytes / (dom_us * 1e-6) / 1e9
        roofline = {"bound": "hbm", "kernel": STAGE_NAME, "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": achieved / peaks["hbm_gbs"], "peak_source": peaks["source"],
                    "frac_of_nominal_8000": achieved / 8000.0,
                    "traffic": None if wl.kind == "stack" else traffic_if_current(wl.name, STAGES[dom]),
                    "algorithmic_bytes_per_launch": wl.alg_bytes}
    roofline["kernel_us_per_launch"] = per_launch_us
    roofline["whole_forward_hbm_frac"] = wl.alg_bytes / (ms_step * 1e-3) / 1e9 / peaks["hbm_gbs"]

    # end to end through the host-pointer entry point: pinned host x -> device -> forward -> pinned host y.
    # Every step does its own two copies; consecutive steps go to different streams (and different handles, each
    # with its own staging buffers), so that one step's upload, another's kernels and a third's download overlap,
    # as a serving loop would run them.  Timed from before the first step's upload to after the last download.
    e2e = None
    if not args.no_e2e:
        nh = min(sets, 4)
        xh = [draw_x(f"xh{rank}_{s}").to(tdt).pin_memory() for s in range(nh)]
        yh = [torch.empty(y_shape, dtype=tdt).pin_memory() for _ in range(nh)]
        lanes = [torch.cuda.Stream() for _ in range(nh)] if nh >= 2 else [stream]   # one stream per (handle, host buffers)

        def forward_host(i):
            hb = sd = i % nh  # a handle, its device staging and its host buffers are only ever used on one stream,
            st = lanes[sd]    # so stream order keeps their reuse safe
            if wl.kind == "stack":   # no host-pointer entry point for stacks: the same copies, issued here
                with torch.cuda.stream(st):
                    xs[sd].copy_(xh[hb], non_blocking=True)
                    circ.circ_stack_forward(stacks[sd], xs[sd], ys[sd], c.batch, st)
                    yh[hb].copy_(ys[sd], non_blocking=True)
            elif wl.kind == "fc":
                circ.circ_fc_forward_host(handles[sd], xh[hb], yh[hb], c.batch, st)
            else:
                circ.circ_conv_forward_host(handles[sd], xh[hb], yh[hb], c.N, c.H, c.W, st)

        for i in range(3):
            forward_host(i)
        torch.cuda.synchronize()
        e2e_steps = min(args.steps, 300)
        if world > 1:
            dist.barrier()
        e0.record(stream)
        for st in lanes:
            st.wait_stream(stream)
        for i in range(e2e_steps):
            forward_host(i)
        for st in lanes:
            stream.wait_stream(st)
        e1.record(stream)
        torch.cuda.synchronize()
        ms_e2e = max_over_ranks(e0.elapsed_time(e1), world)
        e2e = {"value": world * wl.samples * e2e_steps / (ms_e2e * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": int(np.prod(x_shape)) * wl.sx, "d2h_bytes_per_step": int(np.prod(y_shape)) * wl.sy,
               "steps": e2e_steps, "streams": len(lanes)}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        rate, what, threads = oracle_rate(wl)
        cpu = {"value": rate, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": what}

    for st_h in stacks:
        circ.circ_stack_destroy(st_h)
    for h in handles + [hl for hs in stack_layers for hl in hs]:
        circ.circ_destroy(h)
    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if c.bf16_io else "f32", "data": "synthetic",
            "config": {"workload": wl.name, "description": wl.desc, "samples_per_step_per_gpu": wl.samples, "variant": variant, "streams": args.streams,
                       "samples_per_s_with_4_batches_in_flight": overlap4,
                       "l2": f"steps rotate through {sets} distinct (layer, x, y) sets, {sets * per_set / 1e6:.0f} MB > 2 x L2",
                       "dense_equiv_tflops": wl.dense_flops * world / (ms_step * 1e-3) / 1e12},
            "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": int(launches), "clocks": clocks,
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def main() -> int:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20000)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2_b256")
    ap.add_argument("--variant", type=int, default=0, help="force a CIRC_VARIANT_* (0 = planner's choice)")
    ap.add_argument("--max-sets", type=int, default=64)
    ap.add_argument("--streams", type=int, default=1,
                    help="parallel graph branches for independent batches (1 = one forward after another)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
