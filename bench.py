#!/usr/bin/env python
"""Benchmark of the block-circulant forward pass: one JSON line per run.

    python bench.py --gpus N --steps K --warmup W            # the CUDA library (C ABI)
    python bench.py --impl reference --steps K --warmup W    # the fp64 dense CPU oracle
    python bench.py --workload NAME ...                      # another configuration (see workload())

A step is one forward pass of the workload over one batch of seeded synthetic input.  The headline
workload is the largest single-GPU configuration of the benchmark set, the 16384 x 16384, k = 4,
float32 layer at batch 1024; the same JSON line carries a table (`config.table`) with one row per
named configuration and per corner of the n = 16384 sweep.

Timing protocol.  The K steps are captured in a CUDA graph (the GPU, not the host's launch rate, sets
the pace) and rotate through enough distinct (layer, x, y) sets that the working set exceeds twice the
L2 cache, so every byte of every step comes from HBM ("cold").  One repeat = exactly K steps between two
CUDA events; repeats go on until at least 20 of them and half a second have been timed, the L2 is flushed
between repeats, and the MEDIAN repeat is reported.  The "warm" figure is the same with one set and no
flush.  With N > 1 (torchrun, or spawned from here) every rank runs the same job on its own GPU and its
own batches (samples are independent: no collective on the data path); the reported value is all samples
of all ranks divided by the slowest rank's device time.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import math
import os
import re
import socket
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
HEADLINE = "sweep_n16384_k4_b1024"
STAGES = ["input_fft", "contraction", "output_ifft", "fused_fc"]
STAGE_SOURCE = {"input_fft": "circ_staged.cu", "output_ifft": "circ_staged.cu", "contraction": "circ_tensor.cu",
                "fused_fc": "circ_fused.cu"}
TABLE_ROWS = (["cfg1", "cfg2_b1", "cfg2_b16", "cfg2_b256", "cfg3_stack", "cfg4"] +
              [f"sweep_n16384_k{k}_b{b}{d}" for d in ("", "_bf16") for k in (4, 16, 64, 256) for b in (1, 64, 1024)])

# DRAM traffic per launch from ncu captures (dram__bytes_read.sum + dram__bytes_write.sum), keyed by
# (workload, kernel).  Each entry is tied to the sha256 of the kernel's source file at capture time;
# when the source has changed since, the figure is withheld (reported as null).  These are builder-run
# captures (profiles/), not counters read during this run: `traffic_source` in the JSON line says so.
NCU_TRAFFIC: dict = {
    ("sweep_n16384_k4_b1024", "contraction"): {"bytes_per_launch": 616559616, "source_sha256": "92cec56a36476480a1ded93e200f58eb5fed3f5a33f90191daf70a4c15f8f513"},
    ("sweep_n16384_k4_b1", "fused_fc"): {"bytes_per_launch": 272659200, "source_sha256": "b9ba9386726b06f2e3c224c12e7a946d67c050f28211b6514922226939366a3c"},
    ("sweep_n16384_k64_b1024", "contraction"): {"bytes_per_launch": 126377984, "source_sha256": "92cec56a36476480a1ded93e200f58eb5fed3f5a33f90191daf70a4c15f8f513"},
    ("cfg4", "contraction"): {"bytes_per_launch": 13097984, "source_sha256": "92cec56a36476480a1ded93e200f58eb5fed3f5a33f90191daf70a4c15f8f513"},
    ("cfg2_b256", "input_fft"): {"bytes_per_launch": 4212736, "source_sha256": "92670eeeee80adeed252110b54bdb9fa814258a2354f4f6a324b74a2cc8c680a"},
    ("cfg2_b256", "contraction"): {"bytes_per_launch": 6309888, "source_sha256": "92cec56a36476480a1ded93e200f58eb5fed3f5a33f90191daf70a4c15f8f513"},
    ("cfg2_b256", "output_ifft"): {"bytes_per_launch": 4235776, "source_sha256": "92670eeeee80adeed252110b54bdb9fa814258a2354f4f6a324b74a2cc8c680a"},
}


@dataclass
class Workload:
    name: str
    desc: str
    kind: str            # "fc", "stack" or "conv"
    case: object
    samples: int         # samples (FC) or images (CONV) per step
    alg_bytes: int       # bytes the method must move per forward
    dense_flops: float   # flops of the equivalent dense layer per forward
    sx: int
    sy: int
    contraction_flops: float = 0.0   # p q B (4k - 4) (x taps): flops of the per-frequency products
    fft_flops: float = 0.0           # butterflies of the forward and inverse transforms (2.5 k log2 k per real transform)
    spectra_bf16: bool = False       # the streaming kernel reads bfloat16 weight spectra (workload suffix _w16)


_W_CACHE: dict = {}
_X_CACHE: dict = {}


def _sweep_case(n: int, k: int, b: int, bf: bool):
    """Square sweep layer; the defining vectors are drawn once per (n, k) and shared by every batch size and dtype."""
    key = (n, k)
    if key not in _W_CACHE:
        _W_CACHE[key] = synth.normal((n // k, n // k, k), 1.0 / n, synth.stream_id(f"sweep_n{n}_k{k}", "w"))
    xkey = (n, b, "x")
    if xkey not in _X_CACHE:
        _X_CACHE.clear()                                  # one batch shape at a time is enough; keeps the host footprint small
        _X_CACHE[xkey] = synth.uniform((b, n), -1.0, 1.0, synth.stream_id(f"sweep_n{n}_b{b}", "x"))
    x = _X_CACHE[xkey]
    return synth.FcCase(f"sweep_n{n}_k{k}_b{b}_{'bf16' if bf else 'f32'}", n, n, k, b, _W_CACHE[key],
                        synth.round_to_bf16(x) if bf else x, None, False, bf)


def workload(name: str) -> Workload:
    """Named workloads: cfg1, cfg2_b{B}, cfg3_l{0,1,2}, cfg3_stack, cfg4, sweep_n{n}_k{k}_b{B}[_bf16][_w16]."""
    def fft_flops(m, n, k, batch):
        return 2.5 * k * max(1.0, math.log2(k)) * (batch * (m + n) / k)

    def fc(case, desc, w16=False):
        s = 2 if case.bf16_io else 4
        p, q = case.m // case.k, case.n // case.k
        # bytes per stored spectrum value: with bfloat16 activations the tensor-core path (batch > 8, q a multiple of 8)
        # multiplies by, and therefore stores, bfloat16 spectra; every other path reads float32 ones (or _w16's bfloat16)
        s_w = 2 if (w16 or (case.bf16_io and case.batch > 8 and q % 8 == 0)) else 4
        alg = s_w * case.m * case.n // case.k + s * case.batch * (case.n + case.m) + (4 * case.m if case.bias is not None else 0)
        return Workload(name, desc, "fc", case, case.batch, alg, 2.0 * case.m * case.n * case.batch, s, s,
                        float(p) * q * case.batch * (4 * case.k - 4), fft_flops(case.m, case.n, case.k, case.batch), w16)

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
        return fc(_sweep_case(n, k, b, bf),
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
                        sum(float(l.m // l.k) * (l.n // l.k) * 128 * (4 * l.k - 4) for l in layers),
                        sum(fft_flops(l.m, l.n, l.k, 128) for l in layers))
    if name == "cfg4":
        c = synth.config4()
        pix = c.N * c.H * c.W
        alg = 2 * c.r * c.r * c.c_out * c.c_in // c.k + 2 * pix * (c.c_in + c.c_out)     # bfloat16 spectra, bfloat16 pixels
        return Workload(name, "CONV 3x3 pad 1, 256->256 ch, 28x28, batch 32, k=16, bf16 activations", "conv", c, c.N, alg,
                        2.0 * pix * c.r * c.r * c.c_in * c.c_out, 2, 2,
                        float(c.r * c.r) * (c.c_out // c.k) * (c.c_in // c.k) * pix * (4 * c.k - 4),
                        fft_flops(c.c_out, c.c_in, c.k, pix))
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

    def _lines(self) -> int:
        try:
            with open(self.tmp.name) as f:
                return sum(1 for _ in f)
        except OSError:
            return 0

    def start(self, wait_s: float = 5.0):
        """Start sampling and wait until the first samples are on file, so that a short region still has some."""
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                          "-lms", "50", "-i", str(self.index)], stdout=self.tmp, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None
            return
        t0 = time.perf_counter()
        while self._lines() < 2 and time.perf_counter() - t0 < wait_s and self.proc.poll() is None:
            time.sleep(0.05)
        self.lines_before = self._lines()

    def stop(self) -> dict:
        if self.proc is not None:
            time.sleep(0.12)               # let the sampler write the samples of the last 100 ms
            self.proc.terminate()          # the exact child we started
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        self.tmp.flush()
        self.tmp.seek(0)
        sm, smax, reasons = [], [], set()
        for line in self.tmp.read().splitlines()[max(0, getattr(self, "lines_before", 0) - 1):]:
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


def graph_plan(steps: int, cap: int = 256):
    """Split `steps` into (graph length G, replays, remainder): a repeat is `replays` replays of a G-step graph plus
    one replay of a `remainder`-step graph, i.e. exactly `steps` steps."""
    if steps <= cap:
        return steps, 1, 0
    for g in range(cap, 15, -1):
        if steps % g == 0:
            return g, steps // g, 0
    return cap, steps // cap, steps % cap


def sets_needed(per_set_bytes: int, max_sets: int) -> int:
    """Distinct (layer, x, y) sets so that consecutive uses of one set are more than 2 x L2 apart."""
    return int(min(max_sets, max(2, -(-2 * L2_BYTES // max(per_set_bytes, 1)) + 1)))


def own_bytes(wl: Workload, variant: int, circ, s2_kernel: int = 0) -> dict:
    """Bytes each kernel of the path reads and writes itself (its operands), per forward; `s2_kernel` is the
    CIRC_KERNEL_* id of the contraction that ran (it fixes the stored form of the weights and the layout of X)."""
    c = wl.case
    if wl.kind == "stack":
        return {}
    if wl.kind == "fc":
        cols_in = cols_out = 2 * ((c.batch + 1) // 2)
        n, m, taps, k = c.n, c.m, 1, c.k
        x_b, y_b = wl.sx * c.batch * n, wl.sy * c.batch * m
    else:
        nh = (c.N + 1) // 2
        Ho, Wo = c.H + 2 * c.pad - c.r + 1, c.W + 2 * c.pad - c.r + 1
        cols_in, cols_out = 2 * nh * c.H * c.W, 2 * nh * Ho * Wo
        n, m, taps, k = c.c_in, c.c_out, c.r * c.r, c.k
        x_b, y_b = wl.sx * c.N * c.H * c.W * n, wl.sy * c.N * Ho * Wo * m
    if variant == circ.CIRC_VARIANT_FUSED:
        return {"fused_fc": wl.alg_bytes}
    tensor = variant == circ.CIRC_VARIANT_TENSOR
    twin = s2_kernel in (circ.CIRC_KERNEL_S2_TENSOR_TWIN, circ.CIRC_KERNEL_S2_ROWS_TWIN)
    xhat = cols_in * n * (2 if (tensor and c.bf16_io) else 4)          # float32, split bfloat16 (hi + lo), or bfloat16
    if twin:
        xhat = int(xhat * (2.0 - 2.0 / k))                              # the complex problems' columns twice
    yhat = cols_out * m * 4
    spectra = taps * m * n // k                                         # real values of the half spectra
    if tensor:
        part_bytes = 2 if c.bf16_io else 4                              # hi (+ lo) bfloat16
        a_b = spectra * part_bytes if twin else int(spectra * (2.0 - 2.0 / k)) * part_bytes   # embedded [Wr -Wi; Wi Wr]: complex values twice
    else:
        a_b = int(spectra * (2.0 - 2.0 / k)) * 4
    return {"input_fft": x_b + xhat, "contraction": xhat + yhat + a_b, "output_ifft": yhat + y_b}


class Job:
    """One workload on the device: `sets` distinct (layer, x, y) triples and the calls that run a forward on one."""

    def __init__(self, wl: Workload, rank: int, variant: int, max_sets: int, circ, torch):
        self.wl, self.circ, self.torch = wl, circ, torch
        c = wl.case
        self.tdt = torch.bfloat16 if c.bf16_io else torch.float32
        if wl.kind == "fc":
            self.x_shape, self.y_shape = (c.batch, c.n), (c.batch, c.m)
            weight_store = 16 * c.m * c.n // c.k
            workspace = 4 * (c.batch + 1) * (c.m + c.n)
        elif wl.kind == "stack":
            self.x_shape, self.y_shape = (c.batch, c.n), (c.batch, c.m)
            weight_store = sum(16 * l.m * l.n // l.k for l in c.layers)
            workspace = sum(4 * (c.batch + 1) * (l.m + l.n) for l in c.layers)
        else:
            Ho, Wo = c.H + 2 * c.pad - c.r + 1, c.W + 2 * c.pad - c.r + 1
            self.x_shape, self.y_shape = (c.N, c.H, c.W, c.c_in), (c.N, Ho, Wo, c.c_out)
            weight_store = 16 * c.r * c.r * c.c_out * c.c_in // c.k
            workspace = 4 * (c.N + 1) * c.H * c.W * (c.c_in + c.c_out)
        self.per_set = wl.alg_bytes            # only what a forward must touch counts towards the rotation's footprint
        self.sets = sets_needed(self.per_set, max_sets)
        self.footprint_note = (f"steps rotate through {self.sets} distinct (layer, x, y) sets = "
                               f"{self.sets * self.per_set / 1e6:.0f} MB of algorithmic bytes "
                               f"({'>' if self.sets * self.per_set >= 2 * L2_BYTES else 'less than'} 2 x L2); L2 flushed between repeats")
        self.handles, self.xs, self.ys, self.stacks, self.stack_layers = [], [], [], [], []
        x0 = torch.from_numpy(c.x).cuda().to(self.tdt)
        self.create_ms = None      # set 0: create + reserve, i.e. copy of the defining vectors, spectra (S0), stored form, workspace
        for s in range(self.sets):
            if s == 0:
                torch.cuda.synchronize()
                t_create = time.perf_counter()
            elif s == 1:
                torch.cuda.synchronize()
                self.create_ms = 1e3 * (time.perf_counter() - t_create)
            # every set and every rank gets its own batch: the drawn batch, rolled by (rank, set) rows and columns
            xs = x0 if (s == 0 and rank == 0) else torch.roll(x0, shifts=(s + 7 * rank, 3 * s + rank), dims=(0, x0.dim() - 1)).contiguous()
            self.xs.append(xs)
            self.ys.append(torch.empty(self.y_shape, device="cuda", dtype=self.tdt))
            if wl.kind == "stack":
                hs = []
                for l in c.layers:
                    hl = circ.circ_fc_create(l.m, l.n, l.k, l.w)
                    circ.circ_set_activation(hl, int(l.relu))
                    if variant:
                        circ.circ_set_variant(hl, variant)
                    hs.append(hl)
                st_h = circ.circ_stack_create(hs)
                circ.circ_stack_reserve(st_h, c.batch)
                self.stack_layers.append(hs)
                self.stacks.append(st_h)
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
            if variant:
                circ.circ_set_variant(h, variant)
            self.handles.append(h)
        torch.cuda.synchronize()
        if self.create_ms is None:
            self.create_ms = 1e3 * (time.perf_counter() - t_create)

    def first_handle(self):
        return self.stack_layers[0][0] if self.wl.kind == "stack" else self.handles[0]

    def forward(self, s, st, stage=None, times=1):
        c, circ = self.wl.case, self.circ
        if self.wl.kind == "stack":
            circ.circ_stack_forward(self.stacks[s], self.xs[s], self.ys[s], c.batch, st)
        elif stage is not None:
            if self.wl.kind == "fc":
                circ.circ_debug_forward_repeat(self.handles[s], self.xs[s], self.ys[s], c.batch, 1, 1, stage, times, st)
            else:
                circ.circ_debug_forward_repeat(self.handles[s], self.xs[s], self.ys[s], c.N, c.H, c.W, stage, times, st)
        elif self.wl.kind == "fc":
            circ.circ_fc_forward(self.handles[s], self.xs[s], self.ys[s], c.batch, st)
        else:
            circ.circ_conv_forward(self.handles[s], self.xs[s], self.ys[s], c.N, c.H, c.W, st)

    def variant(self) -> int:
        return self.circ.circ_last_variant(self.first_handle())

    def destroy(self):
        for st_h in self.stacks:
            self.circ.circ_stack_destroy(st_h)
        for h in self.handles + [hl for hs in self.stack_layers for hl in hs]:
            self.circ.circ_destroy(h)
        self.handles, self.stacks, self.stack_layers, self.xs, self.ys = [], [], [], [], []


class Timer:
    """Median-of-repeats timing of K-step CUDA graphs on one stream."""

    def __init__(self, torch, circ):
        self.torch, self.circ = torch, circ
        self.stream = torch.cuda.current_stream()
        self.flush_buf = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device="cuda")

    def capture(self, job: Job, steps: int, cold: bool, stage=None, times=1, first_set=0):
        torch = self.torch
        g, cs = torch.cuda.CUDAGraph(), torch.cuda.Stream()
        cs.wait_stream(self.stream)
        l0 = self.circ.circ_debug_launch_count()
        with torch.cuda.graph(g, stream=cs):
            st = torch.cuda.current_stream()
            for i in range(steps):
                job.forward((first_set + i) % job.sets if cold else 0, st, stage, times)
        return g, self.circ.circ_debug_launch_count() - l0

    def time_steps(self, job: Job, steps: int, cold: bool = True, min_s: float = 0.5, min_reps: int = 20, max_s: float = 4.0,
                   stage=None, times=1):
        """Returns (median ms for `steps` steps, repeats timed, kernel launches per repeat)."""
        torch = self.torch
        G, replays, rem = graph_plan(steps)
        main, l_main = self.capture(job, G, cold, stage, times)
        tail, l_tail = (self.capture(job, rem, cold, stage, times, first_set=(G * replays) % max(job.sets, 1)) if rem else (None, 0))

        def one_repeat(e0, e1):
            if cold:
                self.flush_buf.zero_()
            e0.record(self.stream)
            for _ in range(replays):
                main.replay()
            if tail is not None:
                tail.replay()
            e1.record(self.stream)

        # pilot (also a warm-up of the graphs)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        one_repeat(a, b)
        one_repeat(a, b)
        torch.cuda.synchronize()
        t1 = max(a.elapsed_time(b), 1e-3)
        reps = int(min(max(min_reps, math.ceil(1e3 * min_s / t1)), max(min_reps, math.ceil(1e3 * max_s / t1))))
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
        for e0, e1 in evs:
            one_repeat(e0, e1)
        torch.cuda.synchronize()
        times_ms = sorted(e0.elapsed_time(e1) for e0, e1 in evs)
        return float(np.median(times_ms)), reps, l_main * replays + l_tail


def device_floors(torch, circ) -> dict:
    """Box-level reference figures: the float32 FMA rate (micro-benchmark) and the launch floor of an empty kernel."""
    stream = torch.cuda.current_stream()
    blocks, iters = torch.cuda.get_device_properties(torch.cuda.current_device()).multi_processor_count * 8, 8192
    sink = torch.empty(blocks * 256, device="cuda")
    flops = circ.circ_debug_fma_burn(sink, blocks, iters, stream)
    torch.cuda.synchronize()
    best = float("inf")
    for _ in range(5):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        circ.circ_debug_fma_burn(sink, blocks, iters, stream)
        e1.record(stream)
        torch.cuda.synchronize()
        best = min(best, e0.elapsed_time(e1))
    fma_tflops = flops / (best * 1e-3) / 1e12
    # launch floor: 256 empty kernels back to back in one graph
    g, cs = torch.cuda.CUDAGraph(), torch.cuda.Stream()
    cs.wait_stream(stream)
    with torch.cuda.graph(g, stream=cs):
        for _ in range(256):
            circ.circ_debug_empty_kernel(torch.cuda.current_stream())
    g.replay()
    torch.cuda.synchronize()
    ts = []
    for _ in range(20):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        g.replay()
        e1.record(stream)
        torch.cuda.synchronize()
        ts.append(e0.elapsed_time(e1) / 256)
    return {"fp32_fma_tflops": fma_tflops, "launch_floor_us": 1e3 * float(np.median(ts)),
            "how": "circ_debug_fma_burn best of 5; 256 empty kernels per CUDA-graph replay, median of 20"}


def dense_context(torch, m: int, n: int, batch: int) -> dict:
    """torch.matmul of the equivalent dense layer (context only: the O(n^2) work the method avoids, Sec. 3.1)."""
    out = {}
    try:
        for name, dt in (("fp32", torch.float32), ("bf16", torch.bfloat16)):
            w = torch.empty(n, m, device="cuda", dtype=dt).normal_()
            x = torch.empty(batch, n, device="cuda", dtype=dt).normal_()
            prev = torch.backends.cuda.matmul.allow_tf32
            torch.backends.cuda.matmul.allow_tf32 = False
            for _ in range(2):
                torch.matmul(x, w)
            ts = []
            for _ in range(5):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                torch.matmul(x, w)
                e1.record()
                torch.cuda.synchronize()
                ts.append(e0.elapsed_time(e1))
            torch.backends.cuda.matmul.allow_tf32 = prev
            out[f"dense_{name}_us"] = 1e3 * float(np.median(ts))
            del w, x
    except RuntimeError as e:      # not enough memory for the dense matrix: context only, so say so and go on
        out["error"] = str(e)[:120]
    return out


def bound_and_fraction(wl: Workload, variant: int, us: float, peaks: dict, fma_tflops: float, circ) -> dict:
    """Which roofline bounds the whole forward and the fraction of it reached: max(t_hbm, t_compute) / t_measured,
    with the compute time taken on the pipe the chosen variant uses."""
    c = wl.case
    t_hbm = wl.alg_bytes / (peaks["hbm_gbs"] * 1e9)
    tensor = variant == circ.CIRC_VARIANT_TENSOR
    tensor_peak = peaks["bf16_tflops"] / (1.0 if c.bf16_io else 3.0)    # float32 operands: three bfloat16 products
    t_tc = wl.contraction_flops / (tensor_peak * 1e12) if tensor else 0.0
    alu_flops = wl.fft_flops + (0.0 if tensor else wl.contraction_flops)
    t_alu = alu_flops / (fma_tflops * 1e12) if fma_tflops else 0.0
    t = us * 1e-6
    bound, t_bound = max((("hbm", t_hbm), ("tensor", t_tc), ("alu", t_alu)), key=lambda kv: kv[1])
    if bound == "hbm":
        achieved, peak, unit = wl.alg_bytes / t / 1e9, peaks["hbm_gbs"], "GB/s"
    elif bound == "tensor":
        achieved, peak, unit = wl.contraction_flops / t / 1e12, tensor_peak, "TFLOP/s"
    else:
        achieved, peak, unit = alu_flops / t / 1e12, fma_tflops, "TFLOP/s"
    return {"bound": bound, "achieved": achieved, "peak": peak, "unit": unit, "frac": t_bound / t,
            "t_hbm_us": 1e6 * t_hbm, "t_tensor_us": 1e6 * t_tc, "t_alu_us": 1e6 * t_alu}


def run_row(name: str, timer: Timer, peaks: dict, floors: dict, args, circ, torch, rank: int) -> dict:
    """One row of the table: cold and warm time per forward and the whole-forward roofline fraction."""
    wl = workload(name)
    job = Job(wl, rank, 0, args.max_sets, circ, torch)
    try:
        for i in range(3):
            job.forward(i % job.sets, timer.stream)
        torch.cuda.synchronize()
        steps = max(job.sets, 8)
        cold_ms, reps, _ = timer.time_steps(job, steps, cold=True, min_s=args.row_seconds, min_reps=10, max_s=1.0)
        warm_ms, _, _ = timer.time_steps(job, 8, cold=False, min_s=args.row_seconds / 2, min_reps=10, max_s=0.5)
        us = 1e3 * cold_ms / steps
        variant = job.variant()
        rf = bound_and_fraction(wl, variant, us, peaks, floors["fp32_fma_tflops"], circ)
        row = {"workload": name, "path": {1: "fused", 2: "fma", 3: "tensor"}.get(variant, "?"), "us_cold": us,
               "us_warm": 1e3 * warm_ms / 8, "samples_per_s": wl.samples / (us * 1e-6),
               "dense_equiv_tflops": wl.dense_flops / (us * 1e-6) / 1e12, "bound": rf["bound"], "frac": rf["frac"],
               "alg_mb": wl.alg_bytes / 1e6, "repeats": reps, "sets": job.sets,
               "latency_bound": wl.alg_bytes < 32e6, "create_ms": job.create_ms,
               "launch_floors": us / floors["launch_floor_us"]}
        return row
    finally:
        job.destroy()
        torch.cuda.empty_cache()


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

    peaks = measured_peaks()
    timer = Timer(torch, circ)
    stream = timer.stream
    floors = device_floors(torch, circ)

    wl = workload(args.workload)
    c = wl.case
    job = Job(wl, rank, args.variant, args.max_sets, circ, torch)
    warmup = max(args.warmup, 3)
    for i in range(warmup):
        job.forward(i % job.sets, stream)
    torch.cuda.synchronize()
    circ.circ_device_status(job.first_handle())

    # ---- the timed region: repeats of exactly K steps, median reported -------------------------------
    if world > 1:
        dist.barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    torch.cuda.synchronize()
    ms_k, reps, launches_per_repeat = timer.time_steps(job, args.steps, cold=True, min_s=args.seconds, min_reps=20)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    clocks = sampler.stop()
    if clocks["samples"] == 0:
        sys.stderr.write("bench.py: the clock sampler (nvidia-smi) produced no sample during the timed region\n")
        if not args.allow_no_clocks:
            return 3
    ms_k = max_over_ranks(ms_k, world)
    ms_step = ms_k / args.steps
    value = world * wl.samples * args.steps / (ms_k * 1e-3)
    variant = job.variant()
    warm_ms, _, _ = timer.time_steps(job, min(args.steps, 64), cold=False, min_s=0.2, min_reps=10, max_s=1.0)
    warm_us = 1e3 * warm_ms / min(args.steps, 64)

    # ---- per-kernel durations: the same graphs with ONE stage's kernel launched 1 + R times per forward ----
    R = 3
    used_stages = [] if wl.kind == "stack" else [3] if variant == circ.CIRC_VARIANT_FUSED else [0, 1, 2]
    ksteps = max(job.sets, min(args.steps, 32))
    stage_us = {}
    if used_stages:
        base_ms, _, _ = timer.time_steps(job, ksteps, cold=True, min_s=0.25, min_reps=10, max_s=1.5, stage=used_stages[0], times=1)
        for st_i in used_stages:
            rep_ms, _, _ = timer.time_steps(job, ksteps, cold=True, min_s=0.25, min_reps=10, max_s=1.5, stage=st_i, times=1 + R)
            stage_us[STAGES[st_i]] = max(0.0, 1e3 * (rep_ms - base_ms) / (R * ksteps))
    s2_kernel = circ.circ_debug_last_kernels(job.first_handle())[1] if wl.kind != "stack" else 0
    ob = own_bytes(wl, variant, circ, s2_kernel)
    kernels = {}
    for kname, us_k in stage_us.items():
        ent = {"us": us_k, "own_bytes": ob.get(kname), "l2_warm": bool(ob.get(kname, 0) < L2_BYTES)}
        if us_k > 0 and ob.get(kname):
            ent["gbs"] = ob[kname] / (us_k * 1e-6) / 1e9
            ent["frac_of_hbm"] = ent["gbs"] / peaks["hbm_gbs"]
        if kname == "contraction" and variant == circ.CIRC_VARIANT_TENSOR and us_k > 0:
            tp = peaks["bf16_tflops"] / (1.0 if c.bf16_io else 3.0)
            ent["tflops"] = wl.contraction_flops / (us_k * 1e-6) / 1e12
            ent["frac_of_tensor"] = ent["tflops"] / tp
        kernels[kname] = ent

    rf = bound_and_fraction(wl, variant, 1e3 * ms_step, peaks, floors["fp32_fma_tflops"], circ)
    dom = max(stage_us, key=stage_us.get) if stage_us else "whole_stack"
    traffic = traffic_if_current(wl.name, dom) if dom in STAGE_SOURCE else None
    roofline = {"bound": rf["bound"], "achieved": rf["achieved"], "peak": rf["peak"], "unit": rf["unit"], "frac": rf["frac"],
                "scope": "whole forward: max(t_hbm, t_tensor, t_alu) / measured time per step",
                "peak_source": peaks["source"],
                "peak_note": {"hbm": "copy bandwidth", "tensor": "sustained bf16 GEMM rate" + ("" if c.bf16_io else " / 3 (hi*hi + lo*hi + hi*lo)"),
                              "alu": "float32 FMA micro-benchmark of this run"}[rf["bound"]],
                "t_hbm_us": rf["t_hbm_us"], "t_tensor_us": rf["t_tensor_us"], "t_alu_us": rf["t_alu_us"],
                "algorithmic_bytes_per_step": wl.alg_bytes, "contraction_flops_per_step": wl.contraction_flops,
                "hbm_frac_of_measured": wl.alg_bytes / (ms_step * 1e-3) / 1e9 / peaks["hbm_gbs"],
                "hbm_frac_of_nominal_8000": wl.alg_bytes / (ms_step * 1e-3) / 1e9 / 8000.0,
                "kernel": dom, "kernels": kernels, "kernel_ids": (circ.circ_debug_last_kernels(job.first_handle()) if wl.kind != "stack" else None),
                "kernel_frac": (kernels.get(dom, {}).get("frac_of_tensor") if rf["bound"] == "tensor" and dom == "contraction"
                                else kernels.get(dom, {}).get("frac_of_hbm")),
                "kernel_note": "per-kernel durations are differences between graphs with that kernel launched 4x and 1x per forward: "
                               "repeat launches re-read the same buffers, so they are L2-warm where l2_warm is true",
                "traffic": traffic,
                "traffic_source": ("ncu capture of this kernel and workload summarised under profiles/ (dram__bytes_read.sum + "
                                   "dram__bytes_write.sum per launch; not read in this run)") if traffic else None}

    # ---- end to end through the host-pointer entry point: pinned host x -> device -> forward -> pinned host y ----
    # Every step does its own two copies; consecutive steps go to different streams (and different handles, each
    # with its own staging buffers), so that one step's upload, another's kernels and a third's download overlap,
    # as a serving loop would run them.  Timed from before the first step's upload to after the last download.
    e2e = None
    if not args.no_e2e:
        nh = min(job.sets, 4)
        xh = [job.xs[s].cpu().pin_memory() for s in range(nh)]
        yh = [torch.empty(job.y_shape, dtype=job.tdt).pin_memory() for _ in range(nh)]
        lanes = [torch.cuda.Stream() for _ in range(nh)] if nh >= 2 else [stream]   # one stream per (handle, host buffers)

        def forward_host(i):
            hb = sd = i % nh  # a handle, its device staging and its host buffers are only ever used on one stream,
            st = lanes[sd]    # so stream order keeps their reuse safe
            if wl.kind == "stack":   # no host-pointer entry point for stacks: the same copies, issued here
                with torch.cuda.stream(st):
                    job.xs[sd].copy_(xh[hb], non_blocking=True)
                    circ.circ_stack_forward(job.stacks[sd], job.xs[sd], job.ys[sd], c.batch, st)
                    yh[hb].copy_(job.ys[sd], non_blocking=True)
            elif wl.kind == "fc":
                circ.circ_fc_forward_host(job.handles[sd], xh[hb], yh[hb], c.batch, st)
            else:
                circ.circ_conv_forward_host(job.handles[sd], xh[hb], yh[hb], c.N, c.H, c.W, st)

        for i in range(3):
            forward_host(i)
        torch.cuda.synchronize()
        e2e_steps = args.steps
        if world > 1:
            dist.barrier()
        ts, t_begin = [], time.perf_counter()
        while len(ts) < 5 or (time.perf_counter() - t_begin < 0.5 and len(ts) < 200):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for st in lanes:
                st.wait_stream(stream)
            for i in range(e2e_steps):
                forward_host(i)
            for st in lanes:
                stream.wait_stream(st)
            e1.record(stream)
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        ms_e2e = max_over_ranks(float(np.median(ts)), world)
        e2e = {"value": world * wl.samples * e2e_steps / (ms_e2e * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": int(np.prod(job.x_shape)) * wl.sx, "d2h_bytes_per_step": int(np.prod(job.y_shape)) * wl.sy,
               "steps": e2e_steps, "repeats": len(ts), "streams": len(lanes),
               "api": "circ_fc_forward_host" if wl.kind == "fc" else "circ_conv_forward_host" if wl.kind == "conv" else "circ_stack_forward + copies"}

    dense = {}
    if rank == 0 and wl.kind == "fc" and not args.no_dense:
        dense = dense_context(torch, c.m, c.n, c.batch)
    job.destroy()
    torch.cuda.empty_cache()

    table = None
    if rank == 0 and world == 1 and not args.no_table:
        table = []
        for name in TABLE_ROWS:
            try:
                table.append(run_row(name, timer, peaks, floors, args, circ, torch, rank))
            except Exception as e:  # a row that cannot run is reported, not hidden
                table.append({"workload": name, "error": str(e)[:200]})

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        rate, what, threads = oracle_rate(wl)
        cpu = {"value": rate, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": what}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warmup,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if c.bf16_io else "f32", "data": "synthetic",
            "config": {"workload": wl.name, "description": wl.desc, "samples_per_step_per_gpu": wl.samples, "variant": variant,
                       "path": {1: "fused", 2: "fma", 3: "tensor"}.get(variant, "?"),
                       "timing": f"median of {reps} repeats of exactly {args.steps} steps (one CUDA graph per repeat), cold",
                       "l2": job.footprint_note, "create_ms": job.create_ms, "us_per_step_cold": 1e3 * ms_step, "us_per_step_warm": warm_us,
                       "dense_equiv_tflops": wl.dense_flops * world / (ms_step * 1e-3) / 1e12,
                       "floors": floors, "dense_context": dense, "table": table},
            "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e,
            "gpu_launches": int(launches_per_repeat * reps), "launches_per_step": launches_per_repeat / args.steps, "clocks": clocks,
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def spawn_ranks(args) -> int:
    """`--gpus N` without a launcher around it: start N ranks of this script on one node."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), str(Path(__file__).resolve())] + sys.argv[1:]
    return subprocess.call(cmd)


def main() -> int:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=HEADLINE)
    ap.add_argument("--variant", type=int, default=0, help="force a CIRC_VARIANT_* (0 = planner's choice)")
    ap.add_argument("--max-sets", type=int, default=96)
    ap.add_argument("--seconds", type=float, default=0.5, help="minimum timed duration of the headline measurement")
    ap.add_argument("--row-seconds", type=float, default=0.2, help="minimum timed duration of one table row")
    ap.add_argument("--no-table", action="store_true", help="skip config.table (the other configurations)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-dense", action="store_true")
    ap.add_argument("--allow-no-clocks", action="store_true", help="do not fail when nvidia-smi gives no clock sample")
    args = ap.parse_args()
    if args.steps < 1 or args.gpus < 1:
        raise SystemExit("--steps and --gpus must be >= 1")
    if args.impl == "reference":
        return run_reference(args)
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.gpus > 1 and world == 1 and "RANK" not in os.environ:
        return spawn_ranks(args)
    if args.gpus != world:
        sys.stderr.write(f"bench.py: --gpus {args.gpus} but WORLD_SIZE is {world}\n")
        return 2
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
