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
    assert c4.alg_bytes == 4 * 9 * 256 * 256 // 16 + 2 * 32 * 28 * 28 * 512
    s = bench.workload("sweep_n1024_k16_b64_bf16")
    assert s.case.bf16_io and s.sx == 2 and s.case.w.shape == (64, 64, 16)
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
