"""Host-side logic of the benchmark's multi-rank path (replicas only): max-over-ranks timing and the
whole-job aggregate, exercised with two gloo ranks on CPU; plus the oracle leg on a tiny sample."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, {root!r})
import torch.distributed as dist
import bench
rank = int(os.environ["RANK"]); world = int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo")
ms = bench.max_over_ranks(2.0 + 3.0 * rank, world)          # rank 0: 2 ms, rank 1: 5 ms
val = bench.aggregate(1e12, ms, world)
dist.barrier()
if rank == 0:
    print(json.dumps({{"ms": ms, "value": val}}))
dist.destroy_process_group()
"""


def test_two_gloo_ranks_take_the_slowest_time_and_sum_the_work(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
                          "--master-addr", "127.0.0.1", "--master-port", "29611", str(script)],
                         capture_output=True, text=True, env=env, timeout=240)
    assert out.returncode == 0, out.stderr[-2000:]
    line = [l for l in out.stdout.splitlines() if l.startswith("{")][-1]
    d = json.loads(line)
    assert d["ms"] == 5.0
    assert d["value"] == pytest.approx(2 * 1e12 / 5e-3 / 1e12)


def test_single_rank_helpers_and_sample_flops():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, 1) == 3.5
    assert bench.aggregate(2e12, 1.0, 1) == pytest.approx(2000.0)
    W = bench.W
    # one head, all rows: fwd + bwd algorithmic flops of the workload divided by the head count
    assert bench.sample_flops(W.chunk_tokens) * W.heads == pytest.approx(W.fwd_flops() + W.bwd_flops())
    p = bench.measured_peaks()
    assert p["bf16_burst"] > 0 and p["hbm"] > 0 and p["source"] in ("measured", "fallback")


def test_reference_arm_prints_one_json_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0"], capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    d = json.loads(out.stdout.strip().splitlines()[-1])
    assert d["impl"] == "reference" and d["unit"] == "TFLOP/s" and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0


def test_plain_launch_with_gpus_2_starts_two_ranks():
    """`bench.py --gpus 2` started without torchrun must start its two ranks itself; the dry run goes through the
    rendezvous, the max-over-ranks reduction and the aggregate on CPU (gloo) and reports n_gpus = 2."""
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    env["MASTER_PORT"] = "29613"
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--dry-run", "--steps", "1",
                          "--warmup", "0"], capture_output=True, text=True, env=env, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                                   # rank 0 alone prints
    d = json.loads(lines[0])
    assert d["n_gpus"] == 2 and d["dry_run"] is True
    assert d["ms_per_step"] == 3.0                           # the slower rank's time
    sys.path.insert(0, ROOT)
    import bench
    assert d["value"] == pytest.approx(bench.aggregate(bench.W.fwd_flops() + bench.W.bwd_flops(), 3.0, 2))


def test_torchrun_command_uses_the_loopback_address():
    sys.path.insert(0, ROOT)
    import bench
    cmd = bench.torchrun_command(4, ["--gpus", "4"], port=29999)
    assert "--master-addr" in cmd and cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[cmd.index("--nproc-per-node") + 1] == "4" and cmd[-2:] == ["--gpus", "4"]
