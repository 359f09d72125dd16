"""The benchmark's output contract, checked on a short run: one JSON line with the agreed keys."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_default_bench_line_has_the_contract_keys():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--steps", "4", "--warmup", "3",
                          "--no-cpu-baseline"], capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "e2e", "gpu_launches", "clocks", "roofline", "cpu_baseline"):
        assert key in d, key
    assert d["n_gpus"] == 1 and d["steps"] == 4 and d["unit"] == "TFLOP/s" and d["dtype"] == "bf16"
    assert d["value"] > 100 and d["gpu_launches"] == 5 * 4 and d["vs_baseline"] is None
    assert "workload" in d["config"] and "model" not in d["config"]
    r = d["roofline"]
    assert r["bound"] == "tensor" and 0 < r["frac"] < 1.2 and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    e = d["e2e"]
    assert e["value"] > 0 and e["h2d_bytes_per_step"] == 4 * 4680 * 12 * 128 * 2
    assert e["d2h_bytes_per_step"] == 4 * 4680 * 12 * 128 * 2 + 12 * 4680 * 4
    assert set(d["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}
    # a 4-step region is far below a second: the burst figure is the denominator, the other fraction is beside it
    assert "burst" in r["peak_source"] and r["frac"] == pytest.approx(r["frac_of_burst"])
    assert r["traffic"] is None or r["traffic"] > 1e8
    # both halves of the metric and their neighbours are timed in the same run
    ro = d["rollout"]
    assert ro["metric"] == "rollout_latent_frames_per_s" and ro["value"] > 0 and ro["chunks"] == 16
    assert ro["append"]["bytes_moved"] == 2 * 2 * 4 * 12 * 3 * 1560 * 128 * 2 and 0 < ro["append"]["frac_of_hbm"] < 1.2
    assert d["rl_update"]["fwd"]["tflops"] > 100 and d["rl_update"]["bwd"]["tflops"] > 100
    assert [(v["attended_frames"], v["chunk_frames"]) for v in d["window_variants"]] == [(21, 3), (21, 1), (15, 3), (15, 1)]
    assert 0.5 < d["score_sensitivity"]["slowdown_x8"] < 2.0
