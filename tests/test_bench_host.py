"""Host-side logic of bench.py that needs no GPU: workload table, byte / flop accounting, the
max-over-ranks reduction on a 2-rank gloo group, the reference arm's JSON line."""
import json
import os
import subprocess
import sys
from pathlib import Path

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parent.parent
sys.path.insert(0, str(ROOT))
import bench  # noqa: E402


def test_workload_accounting():
    w = bench.workload("cfg2_b256")
    # 4 m n / k + 4 B (n + m) + 4 m  (stored spectra + x + y + bias)
    assert w.alg_bytes == 4 * 4096 * 4096 // 64 + 4 * 256 * 8192 + 4 * 4096 == 9453568
    assert w.contraction_flops == 64 * 64 * 256 * (4 * 64 - 4)
    assert w.dense_flops == 2.0 * 4096 * 4096 * 256 and w.samples == 256
    c4 = bench.workload("cfg4")
    assert c4.kind == "conv" and c4.samples == 32
    assert c4.alg_bytes == 2 * 9 * 256 * 256 // 16 + 2 * 32 * 28 * 28 * 512      # bfloat16 spectra and pixels
    s = bench.workload("sweep_n1024_k16_b64_bf16")
    assert s.case.bf16_io and s.sx == 2 and s.case.w.shape == (64, 64, 16)
    # bfloat16 activations on the tensor path: the stored spectra are bfloat16 too; the one-launch kernel reads float32 ones
    assert s.alg_bytes == 2 * 1024 * 1024 // 16 + 2 * 64 * 2048
    assert bench.workload("sweep_n1024_k16_b1_bf16").alg_bytes == 4 * 1024 * 1024 // 16 + 2 * 1 * 2048
    assert bench.workload("sweep_n1024_k256_b64_bf16").alg_bytes == 4 * 1024 * 1024 // 256 + 2 * 64 * 2048   # q = 4: FMA path
    l2 = bench.workload("cfg3_l2")
    assert (l2.case.m, l2.case.n, l2.case.k, l2.case.batch) == (1024, 4096, 128, 128) and l2.case.x.shape == (128, 4096)
    with pytest.raises(SystemExit):
        bench.workload("nope")


def test_traffic_is_withheld_when_the_kernel_changed(monkeypatch):
    src = ROOT / "paper_1708_08917_b200" / "csrc" / "circ_fused.cu"
    import hashlib
    good = hashlib.sha256(src.read_bytes()).hexdigest()
    monkeypatch.setattr(bench, "NCU_TRAFFIC", {("w", "fused_fc"): {"bytes_per_launch": 123, "source_sha256": good}})
    assert bench.traffic_if_current("w", "fused_fc") == 123
    monkeypatch.setattr(bench, "NCU_TRAFFIC", {("w", "fused_fc"): {"bytes_per_launch": 123, "source_sha256": "0" * 64}})
    assert bench.traffic_if_current("w", "fused_fc") is None
    assert bench.traffic_if_current("other", "fused_fc") is None


def test_graph_plan_times_exactly_the_requested_steps():
    for steps in (1, 20, 256, 257, 300, 2000, 20000, 1009):
        g, replays, rem = bench.graph_plan(steps)
        assert g * replays + rem == steps and 1 <= g <= 256 and 0 <= rem < g


def test_rotation_covers_twice_the_l2():
    assert bench.sets_needed(403_000_000, 96) == 2
    assert bench.sets_needed(9_453_568, 96) * 9_453_568 >= 2 * bench.L2_BYTES
    assert bench.sets_needed(18_000, 96) == 96                       # capped: the flush between repeats covers the rest


def test_table_lists_every_named_configuration_and_the_sweep_corners():
    rows = bench.TABLE_ROWS
    assert len(rows) >= 20 and len(set(rows)) == len(rows)
    for must in ("cfg1", "cfg2_b1", "cfg2_b16", "cfg2_b256", "cfg3_stack", "cfg4", "sweep_n16384_k4_b1", "sweep_n16384_k256_b1024_bf16"):
        assert must in rows
    assert bench.HEADLINE == "sweep_n16384_k4_b1024"


def test_whole_forward_fraction_rule():
    class Ids:
        CIRC_VARIANT_FUSED, CIRC_VARIANT_STAGED, CIRC_VARIANT_TENSOR = 1, 2, 3
    peaks = {"hbm_gbs": 6500.0, "bf16_tflops": 1400.0, "source": "test"}
    w = bench.workload("cfg2_b256")
    # tensor path, HBM-bound by the rule: fraction = t_hbm / t
    t_hbm_us = w.alg_bytes / 6500e9 * 1e6
    r = bench.bound_and_fraction(w, 3, 10.0, peaks, 70.0, Ids)
    assert r["bound"] == "hbm" and abs(r["frac"] - t_hbm_us / 10.0) < 1e-9
    assert abs(r["achieved"] - w.alg_bytes / 10e-6 / 1e9) < 1e-6 and r["peak"] == 6500.0
    # the same layer on the FMA pipes is bound by float32 arithmetic
    r = bench.bound_and_fraction(w, 2, 10.0, peaks, 70.0, Ids)
    assert r["bound"] == "alu" and r["t_alu_us"] > r["t_hbm_us"]
    # float32 inputs take three bfloat16 products: a third of the tensor peak
    big = bench.Workload("x", "", "fc", w.case, 1024, 403_000_000, 5.5e14, 4, 4, 2.06e11, 1e9)
    r = bench.bound_and_fraction(big, 3, 500.0, peaks, 70.0, Ids)
    assert r["bound"] == "tensor" and abs(r["peak"] - 1400.0 / 3) < 1e-9
    assert abs(r["frac"] - (2.06e11 / (1400e12 / 3)) / 500e-6) < 1e-9


def test_gpus_flag_must_match_the_launch(monkeypatch):
    monkeypatch.setenv("WORLD_SIZE", "2")
    monkeypatch.setenv("RANK", "0")
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "4"])
    assert bench.main() == 2                                         # --gpus 4 inside a 2-rank launch: refused


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    got = bench.max_over_ranks(10.0 + 5.0 * rank, world)       # rank 0: 10 ms, rank 1: 15 ms
    out.put((rank, got))
    dist.destroy_process_group()


def test_max_over_ranks_world_size_2_gloo():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = dict(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res == {0: 15.0, 1: 15.0}                           # every rank sees the slowest rank's time
    assert bench.max_over_ranks(7.0, 1) == 7.0


def test_reference_arm_prints_one_json_line():
    env = dict(os.environ, OMP_NUM_THREADS="4")
    out = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--steps", "2", "--warmup", "1",
                          "--workload", "cfg1"], capture_output=True, text=True, env=env, timeout=300)
    assert out.returncode == 0, out.stderr
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["unit"] == "samples/s" and d["cpu_baseline"]["kind"] == "oracle"
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["gpu_launches"] == 0 and d["value"] > 0
    # other ranks of a multi-rank launch print nothing and exit 0
    env["RANK"] = "1"
    out = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0"],
                         capture_output=True, text=True, env=env, timeout=120)
    assert out.returncode == 0 and out.stdout.strip() == ""
