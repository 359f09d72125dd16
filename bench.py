#!/usr/bin/env python
"""Benchmark of rolling-KV chunk attention on the single-layer 1.3B-class shape.

One step = one pass of the whole hot path on one batch of synthetic input:
evict 3 frames, forward (O, LSE) of a 3-frame chunk (4680 queries) against 18 held
frames + the chunk (32760 keys), backward (delta, dQ, dK/dV of the chunk), append the
chunk's K/V.  12 heads, head_dim 128, 1560 tokens per latent frame, bf16, scale 1/sqrt(D).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line.  With N > 1 every rank runs an independent replica of the step on
its own GPU (the path has no exchange step); the time is the maximum over ranks and the
value the sum of the work.  Started plainly with --gpus N > 1 the script starts its N
ranks itself through torch.distributed.run.  At N = 1 the line also carries sub-records
for a short streaming rollout (latent-frames/s), the clip-window update, the window
presets and the forward's sensitivity to peaky scores.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

from paper_2603_17051_b200 import synth

METRIC = "chunk_attn_fwd_bwd_tflops"
UNIT = "TFLOP/s"
W = synth.LAYER_FWD
WORKLOAD = ("layer_fwd shape + backward: B=1 H=12 D=128 T=1560, chunk 3 frames (4680 q), 18 held frames + chunk = "
            "32760 keys, S=3 sink + 18 window slots; step = evict 3, fwd, bwd (delta+dQ+dK/dV), append 3")


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"bf16_burst": float(p["bf16_tflops"]), "bf16_sustained": float(p["bf16_tflops_sustained"]),
                "hbm": float(p["hbm_gbs"]), "source": "measured"}
    return {"bf16_burst": 1590.0, "bf16_sustained": 1400.0, "hbm": 6650.0, "source": "fallback"}


def rank_env():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def torchrun_command(n_gpus: int, argv, port: int = 29511):
    """The command that starts one rank per GPU on this node (rendezvous on 127.0.0.1)."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(int(n_gpus)),
            "--master-addr", "127.0.0.1", "--master-port", str(int(port)), os.path.abspath(__file__)] + list(argv)


def relaunch_under_torchrun(args, argv) -> int:
    """`bench.py --gpus N` started plainly (no WORLD_SIZE in the environment): start N ranks of this script."""
    port = int(os.environ.get("MASTER_PORT", "29511"))
    return subprocess.call(torchrun_command(args.gpus, argv, port))


def source_digest(names) -> str:
    """SHA-1 over the named kernel sources: a counter file is only valid for the sources it was taken from."""
    import hashlib
    h = hashlib.sha1()
    for n in names:
        with open(os.path.join(ROOT, "paper_2603_17051_b200", "csrc", n), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def ncu_traffic():
    """DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the attention kernels on the layer
    shape, from the text summary of the ncu capture under profiles/.  An entry is None when the file is missing or
    was taken from other kernel sources than the ones in the tree."""
    out = {"fwd": None, "dq": None, "dkv": None}
    path = os.path.join(ROOT, "profiles", "dram_traffic_layer_shape.txt")
    if not os.path.exists(path):
        return out
    digests = {"fwd": source_digest(["attn_fwd.cuh", "attn_common.cuh", "sm100_ptx.cuh"]),
               "dq": source_digest(["attn_bwd.cuh", "attn_common.cuh", "sm100_ptx.cuh"])}
    digests["dkv"] = digests["dq"]
    with open(path) as f:
        for line in f:
            parts = line.split()
            if len(parts) == 3 and parts[0] in out and parts[2] == digests[parts[0]]:
                out[parts[0]] = float(parts[1])
    return out


def max_over_ranks(value: float, world: int, device=None) -> float:
    """Largest value any rank holds (the job is as slow as its slowest rank)."""
    if world == 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate(flops_per_rank_step: float, ms_per_step_max: float, world: int) -> float:
    """Whole-job TFLOP/s of `world` independent replicas whose slowest one takes ms_per_step_max."""
    return world * flops_per_rank_step / (ms_per_step_max * 1e-3) / 1e12


class ClockSampler:
    """Samples SM clocks and throttle reasons of one GPU with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap,power.draw,power.limit")
    NAMES = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")

    def __init__(self, gpu_id: str):
        self.gpu_id = gpu_id
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", self.gpu_id, "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "50"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.06)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        mhz, mx, reasons, watts, limit = [], None, set(), [], None
        for ts, line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 6 or not (t0 <= ts <= t1 + 0.05):
                continue
            try:
                mhz.append(float(parts[0])); mx = float(parts[1])
            except ValueError:
                continue
            try:
                watts.append(float(parts[6])); limit = float(parts[7])
            except (ValueError, IndexError):
                pass
            for name, val in zip(self.NAMES, parts[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not mhz:  # region shorter than the sampling period: take whatever was seen
            for ts, line in self.lines:
                parts = [p.strip() for p in line.split(",")]
                try:
                    mhz.append(float(parts[0])); mx = float(parts[1])
                except (ValueError, IndexError):
                    pass
        return {"sm_mhz": float(np.median(mhz)) if mhz else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(mhz), "power_w": float(np.median(watts)) if watts else None, "power_limit_w": limit}


# ----------------------------------------------------------------------------------------------- CPU oracle leg
def oracle_sample_inputs(n_rows: int):
    """One head of the workload, `n_rows` query rows: bf16-rounded N(0,1) widened to fp64."""
    from oracle import rolling_attn as orc
    D = W.head_dim
    mk = lambda i, n: orc.bf16_bits_to_f64(synth.normal_bf16(synth.tensor_seed(2, 900 + i), (1, n, 1, D)))
    return (mk(0, n_rows), mk(1, W.ctx_tokens), mk(2, W.ctx_tokens), mk(3, W.chunk_tokens), mk(4, W.chunk_tokens),
            mk(5, n_rows))


def oracle_step(inp):
    from oracle import rolling_attn as orc
    q, kx, vx, kc, vc, do = inp
    o, lse = orc.chunk_attn_fwd(q, kx, vx, kc, vc, W.scale)
    orc.bwd_delta(o, do)
    return orc.chunk_attn_bwd(q, kx, vx, kc, vc, do, W.scale)


def sample_flops(n_rows: int) -> float:
    D, nk, nkc = W.head_dim, W.total_keys, W.chunk_tokens
    return n_rows * D * (4.0 * nk + 6.0 * nk + 4.0 * nkc)


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return int(max(n)) if n else (os.cpu_count() or 1)
    except Exception:
        return os.cpu_count() or 1


def time_oracle(n_rows: int, reps: int):
    inp = oracle_sample_inputs(n_rows)
    t0 = time.perf_counter()
    for _ in range(reps):
        oracle_step(inp)
    dt = (time.perf_counter() - t0) / reps
    return sample_flops(n_rows) / dt / 1e12, dt


def run_reference(args):
    """The CPU oracle as it stands, timed on the host cores, on a bounded sample of the same workload."""
    rank, _, world = rank_env()
    if rank != 0:
        return 0
    n_rows = 256
    sample = "1 of 12 heads x %d of 4680 query rows against all 32760 keys, fwd+bwd, fp64 numpy" % n_rows
    inp = oracle_sample_inputs(n_rows)
    for _ in range(args.warmup):
        oracle_step(inp)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(inp)
    dt = (time.perf_counter() - t0) / max(args.steps, 1)
    val = sample_flops(n_rows) / dt / 1e12
    cores = blas_threads()
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "note": "each step is the bounded sample below, not the whole workload"},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


# ----------------------------------------------------------------------------------------------- GPU arm
def run_dry(args):
    """The multi-rank plumbing without a GPU: rendezvous (gloo), max-over-ranks timing, whole-job aggregate and the
    JSON line of rank 0, with a made-up step time.  Used to check the launch path on a CPU-only machine."""
    import torch.distributed as dist
    rank, _, world = rank_env()
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("gloo")
    ms_step = max_over_ranks(2.0 + rank, world)
    value = aggregate(W.fwd_flops() + W.bwd_flops(), ms_step, world)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps({"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                          "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
                          "dry_run": True, "data": "none (launch-path check, made-up step time)"}))
    return 0


def run_ours(args):
    import torch
    from paper_2603_17051_b200 import binding as A

    rank, local_rank, world = rank_env()
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    dev = torch.device("cuda", local_rank if world > 1 else 0)
    torch.cuda.set_device(dev)
    peaks = measured_peaks()
    B, H, D, T, M = W.batch, W.heads, W.head_dim, W.tokens_per_frame, W.chunk_tokens
    c = W.chunk_frames

    def host_normal(i, shape):
        bits = synth.normal_bf16(synth.tensor_seed(2, 100 * rank + i), shape)
        return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16)

    # inputs: resident copies for the device-timed arm, pinned host copies for the end-to-end arm
    h_q, h_kc, h_vc, h_do = (host_normal(i, (B, M, H, D)).pin_memory() for i in range(4))
    q, kc, vc, do = (t.to(dev) for t in (h_q, h_kc, h_vc, h_do))
    cache = A.astro_kvcache_create(W.cache_batch, H, D, T, W.sink_frames, W.window_frames, device=dev)
    fill = W.held_frames + c                                 # start full: every step evicts 3 then appends 3
    kfill = host_normal(10, (W.cache_batch, fill * T, H, D)).to(dev)
    vfill = host_normal(11, (W.cache_batch, fill * T, H, D)).to(dev)
    A.astro_kvcache_append(cache, kfill, vfill, fill)
    del kfill, vfill
    delta = torch.empty((B, H, M), dtype=torch.float32, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)     # > 126 MB L2
    scale = W.scale

    def make_set(src=None):
        """Device buffers of one step: inputs (copies of `src` or fresh) and outputs."""
        ins = [t.clone() for t in src] if src is not None else [torch.empty_like(q) for _ in range(4)]
        outs = [torch.empty_like(q), torch.empty((B, H, M), dtype=torch.float32, device=dev), torch.empty_like(q),
                torch.empty_like(q), torch.empty_like(q)]                       # o, lse, dq, dk, dv
        return ins, outs
    main_set = ([q, kc, vc, do], make_set()[1])

    def step(ev=None, bufs=None):
        """One pass of the hot path on device buffers; `ev` collects (name, start, end) events per stage."""
        (q_, kc_, vc_, do_), (o_, lse_, dq_, dk_, dv_) = bufs if bufs is not None else main_set
        def stage(name, fn):
            if ev is None:
                fn(); return
            s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            s.record(); fn(); e.record(); ev.append((name, s, e))
        A.astro_kvcache_evict(cache, c)
        stage("fwd", lambda: A.astro_chunk_attn_fwd(cache, q_, kc_, vc_, scale, o=o_, lse=lse_))
        stage("delta", lambda: A.astro_chunk_attn_bwd_delta(o_, do_, delta=delta))
        stage("dq", lambda: A.astro_chunk_attn_bwd_dq(cache, q_, kc_, vc_, lse_, delta, do_, scale, dq=dq_))
        stage("dkv", lambda: A.astro_chunk_attn_bwd_dkv(q_, kc_, vc_, lse_, delta, do_, scale, dk_chunk=dk_, dv_chunk=dv_))
        stage("append", lambda: A.astro_kvcache_append(cache, kc_, vc_, c))
    launches_per_step = 5

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()

    # ---- device-timed region: K steps, each bracketed by its own events, L2 flushed between steps
    gpu_id = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid).replace("GPU-", "")
    sampler = ClockSampler(gpu_id)
    sampler.start()
    time.sleep(0.12)
    barrier()
    t_wall0 = time.time()
    step_events, stage_events = [], []
    for _ in range(args.steps):
        flush.zero_()
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s.record(); step(stage_events); e.record()
        step_events.append((s, e))
    barrier()
    t_wall1 = time.time()
    clocks = sampler.stop(t_wall0, t_wall1)
    ms_step_local = float(np.mean([s.elapsed_time(e) for s, e in step_events]))
    stage_ms = {}
    for name, s, e in stage_events:
        stage_ms.setdefault(name, []).append(s.elapsed_time(e))
    stage_ms = {k: float(np.mean(v)) for k, v in stage_ms.items()}
    A.astro_last_device_status()
    ms_step = max_over_ranks(ms_step_local, world, dev)
    flops_step = W.fwd_flops() + W.bwd_flops()
    value = aggregate(flops_step, ms_step, world)

    # ---- end to end: the same step through the public API with host buffers.  Every step copies its inputs from
    #      pinned host memory and its results back, all inside the timed region; two buffer sets and two copy
    #      streams let the copies of neighbouring steps overlap the kernels of the current one.
    h_in = (h_q, h_kc, h_vc, h_do)
    h_out = [torch.empty((B, M, H, D), dtype=torch.bfloat16).pin_memory(), torch.empty((B, H, M), dtype=torch.float32).pin_memory()]
    h_out += [torch.empty((B, M, H, D), dtype=torch.bfloat16).pin_memory() for _ in range(3)]
    h2d = sum(t.numel() * t.element_size() for t in h_in)
    d2h = sum(t.numel() * t.element_size() for t in h_out)
    sets = [make_set(), make_set()]
    main = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    ev_in = [torch.cuda.Event() for _ in range(2)]      # inputs of the set are on the device
    ev_done = [torch.cuda.Event() for _ in range(2)]    # kernels of the set have finished
    ev_out = [torch.cuda.Event() for _ in range(2)]     # results of the set are on the host

    def e2e_steps(n):
        for i in range(n):
            ins, outs = sets[i & 1]
            with torch.cuda.stream(s_in):
                if i >= 2:
                    s_in.wait_event(ev_done[i & 1])      # the kernels of step i-2 no longer read these inputs
                for d_t, h_t in zip(ins, h_in):
                    d_t.copy_(h_t, non_blocking=True)
                ev_in[i & 1].record(s_in)
            main.wait_event(ev_in[i & 1])
            if i >= 2:
                main.wait_event(ev_out[i & 1])           # the results of step i-2 have left these buffers
            step(bufs=sets[i & 1])
            ev_done[i & 1].record(main)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_done[i & 1])
                for h_t, d_t in zip(h_out, outs):
                    h_t.copy_(d_t, non_blocking=True)
                ev_out[i & 1].record(s_out)
        main.wait_stream(s_out)
        main.wait_stream(s_in)
    e2e_steps(4)
    barrier()
    n_e2e = max(4, min(args.steps, 50))
    s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s.record()
    e2e_steps(n_e2e)
    e.record()
    barrier()
    ms_e2e = max_over_ranks(s.elapsed_time(e) / n_e2e, world, dev)
    e2e_value = aggregate(flops_step, ms_e2e, world)

    if rank != 0:
        if world > 1:
            torch.distributed.destroy_process_group()
        return 0

    # ---- roofline of the dominant kernel (largest share of the step), timed live above
    kernel_flops = {"fwd": ("chunk_attn_fwd_kernel<128>", W.fwd_flops()),
                    "dq": ("chunk_attn_bwd_dq_kernel<128>", 6.0 * B * H * M * W.total_keys * D),
                    "dkv": ("chunk_attn_bwd_dkv_kernel<128>", 4.0 * B * H * M * M * D)}
    dom = max(kernel_flops, key=lambda k: stage_ms[k])
    kname, kflops = kernel_flops[dom]
    achieved = kflops / (stage_ms[dom] * 1e-3) / 1e12
    # A short timed region runs at burst clocks, a longer one settles at the board's power limit: compare with the
    # cuBLAS figure measured in the same regime, and give the other fraction beside it.  The regime is read off the
    # clocks sampled during the region (power cap active and the median SM clock under 90 % of its maximum: the
    # region ran power-capped, however short it was); without samples, off its length.
    timed_s = (t_wall1 - t_wall0)
    capped = ("sw_power_cap" in (clocks.get("reasons") or [])) and \
        (clocks.get("sm_mhz") or 0) < 0.9 * (clocks.get("sm_max_mhz") or 1e9)
    regime = "sustained" if (timed_s >= 1.0 or capped) else "burst"
    peak = peaks["bf16_" + regime]
    traffic = ncu_traffic()
    roofline = {"bound": "tensor", "kernel": kname, "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                "frac": achieved / peak, "traffic": traffic[dom], "traffic_unit": "bytes of DRAM traffic per launch",
                "peak_source": "%s cuBLAS bf16 %s figure (timed region %.2f s, SM clock median %s MHz%s); burst %.1f, "
                               "sustained %.1f" % (peaks["source"], regime, timed_s, clocks.get("sm_mhz"),
                                                   ", power cap active" if capped else "", peaks["bf16_burst"],
                                                   peaks["bf16_sustained"]),
                "frac_of_burst": achieved / peaks["bf16_burst"], "frac_of_sustained": achieved / peaks["bf16_sustained"],
                "frac_of_nominal_2250": achieved / 2250.0, "ms_per_launch": stage_ms[dom],
                "algorithmic_flops_per_launch": kflops}
    per_kernel = {}
    for k, (name, fl) in kernel_flops.items():
        t = fl / (stage_ms[k] * 1e-3) / 1e12
        per_kernel[k] = {"kernel": name, "ms": stage_ms[k], "tflops": t, "frac_of_sustained": t / peaks["bf16_sustained"],
                         "frac_of_burst": t / peaks["bf16_burst"], "dram_bytes_per_launch": traffic[k]}
    bwd_ms = stage_ms["delta"] + stage_ms["dq"] + stage_ms["dkv"]
    per_kernel["bwd_total"] = {"ms": bwd_ms, "tflops": W.bwd_flops() / (bwd_ms * 1e-3) / 1e12}
    append_bytes = 2 * 2 * W.cache_batch * H * c * T * D * 2
    per_kernel["append"] = {"kernel": "ring_copy_kernel<true>", "ms": stage_ms["append"],
                            "gbs": append_bytes / (stage_ms["append"] * 1e-3) / 1e9,
                            "frac_of_hbm": append_bytes / (stage_ms["append"] * 1e-3) / 1e9 / peaks["hbm"]}
    per_kernel["delta"] = {"kernel": "bwd_delta_kernel<128>", "ms": stage_ms["delta"]}

    # ---- the other half of the metric and its neighbours, as sub-records (one GPU only): a short streaming rollout
    #      (latent-frames/s), the clip-window update (forward + backward TFLOP/s), the per-frame / 15-frame window
    #      presets and the forward's sensitivity to peaky scores
    legs = {}
    if world == 1 and not args.no_legs:
        del cache, flush
        torch.cuda.empty_cache()
        legs["rollout"] = measure_rollout(A, dev, peaks, chunks=args.rollout_chunks, reading="A")
        legs["rl_update"] = measure_rl_update(A, dev, peaks, reps=10)
        legs["window_variants"] = measure_variants(A, dev, peaks, reps=10)
        legs["score_sensitivity"] = measure_score_sensitivity(A, dev, peaks, reps=10)

    # ---- CPU oracle on a bounded sample (rank 0, N = 1 only)
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        n_rows = 4680
        v_cpu, dt = time_oracle(n_rows, 1)
        cpu = {"value": v_cpu, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "seconds": dt,
               "sample": "1 of 12 heads, all 4680 query rows x 32760 keys, fwd+bwd once, fp64 numpy"}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic", "config": {"workload": WORKLOAD, "l2": "flushed between timed steps (256 MB write)",
                                            "timing": "CUDA events per step, mean over steps, max over ranks",
                                            "parallelism": "replicas only (no exchange step)",
                                            "e2e": "every step copies its inputs from pinned host memory and its results "
                                                   "back inside the timed region; two buffer sets and two copy streams "
                                                   "overlap those copies with the kernels; no L2 flush in that loop"},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "ms_per_step": ms_e2e},
            "gpu_launches": launches_per_step * args.steps, "clocks": clocks, "roofline": roofline,
            "cpu_baseline": cpu, "kernels": per_kernel}
    line.update(legs)
    print(json.dumps(line))
    if world > 1:
        torch.distributed.destroy_process_group()
    return 0


# ----------------------------------------------------------------------------------------------- other workloads
def _event_ms(fn, reps=1):
    import torch
    s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    s.record()
    for _ in range(reps):
        fn()
    e.record()
    torch.cuda.synchronize()
    return s.elapsed_time(e) / reps


# ----------------------------------------------------------------------------------------------- workload legs
def _rnd(dev, i, shape):
    import torch
    bits = synth.normal_bf16(synth.tensor_seed(9, i), shape)
    return torch.from_numpy(bits.view(np.int16)).to(dev).view(torch.bfloat16)


def measure_rollout(A, dev, peaks, chunks=80, reading="A", steps=4):
    """Streaming rollout (B = 4 per-sample caches, 3 sink + 12 window slots, 3-frame chunks): per chunk evict,
    `steps` denoising-step forwards against the fixed cache, one clean K/V append.  One stream, CUDA events."""
    import torch
    w = synth.ROLLOUT
    H, D, T, c, B = w.heads, w.head_dim, w.tokens_per_frame, w.chunk_frames, w.batch
    M = c * T
    slots = w.window_frames if reading == "A" else w.window_frames + c
    cache = A.astro_kvcache_create(B, H, D, T, w.sink_frames, slots, device=dev)
    q, kc, vc = (_rnd(dev, i, (B, M, H, D)) for i in range(3))
    o = torch.empty_like(q); lse = torch.empty((B, H, M), dtype=torch.float32, device=dev)
    cap = w.sink_frames + slots

    def rollout(n_chunks):
        A.astro_kvcache_reset(cache)
        flops = 0.0
        for n in range(n_chunks):
            sink, win, _ = A.astro_kvcache_query(cache)
            over = sink + win - (cap - c)
            if over > 0:
                A.astro_kvcache_evict(cache, over)
            held = min(sink + win, cap - c)
            for _ in range(steps):                       # denoising steps against a fixed cache
                A.astro_chunk_attn_fwd(cache, q, kc, vc, w.scale, o=o, lse=lse)
            flops += steps * 4.0 * B * H * M * (held * T + M) * D
            A.astro_kvcache_append(cache, kc, vc, c)     # one clean-frame K/V write
        return flops
    rollout(min(chunks, 6))
    torch.cuda.synchronize()
    s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s.record(); flops = rollout(chunks); e.record(); torch.cuda.synchronize()
    ms = s.elapsed_time(e)
    A.astro_last_device_status()
    frames = chunks * c
    # append alone: 3 frames of K and V for all samples, read + written once.  16 (evict, append) pairs back to back
    # from four rotating source buffers (460 MB, larger than L2), so that neither the launch gap after a
    # synchronise nor L2 hits on the source enter the figure
    srcs = [(kc, vc)] + [(torch.empty_like(kc).copy_(kc), torch.empty_like(vc).copy_(vc)) for _ in range(3)]
    def appends(n):
        for i in range(n):
            A.astro_kvcache_evict(cache, c)
            A.astro_kvcache_append(cache, srcs[i & 3][0], srcs[i & 3][1], c)
    appends(4)
    app_ms = _event_ms(lambda: appends(16)) / 16
    del srcs
    app_bytes = 2 * 2 * B * H * c * T * D * 2
    tf = flops / (ms * 1e-3) / 1e12
    regime = "burst" if ms < 1000.0 else "sustained"
    return {"workload": "rollout", "reading": reading, "chunks": chunks, "denoising_steps": steps,
            "append": {"kernel": "ring_copy_kernel<true>", "ms": app_ms, "bytes_moved": app_bytes,
                       "gbs": app_bytes / app_ms / 1e6, "frac_of_hbm": app_bytes / app_ms / 1e6 / peaks["hbm"]},
            "metric": "rollout_latent_frames_per_s", "value": frames * B / (ms * 1e-3),
            "unit": "latent-frames/s (all %d samples, attention of one layer)" % B,
            "per_sample_latent_frames_per_s": frames / (ms * 1e-3), "ms_total": ms, "tflops": tf,
            "keys_steady_state": (cap - c) * T + M,
            "config": "B=4 H=12 D=128 T=1560, S=3 + %d window slots, %d chunks x (evict, %d fwd, append)" % (slots, chunks, steps),
            "frac_of_bf16_%s" % regime: tf / peaks["bf16_" + regime]}


def measure_rl_update(A, dev, peaks, reps=20):
    """Clip-window update: B = 2, 28080 detached context keys + 4680 trainable queries/keys; forward with LSE, then
    backward (delta, dQ over all keys, dK/dV of the chunk)."""
    import torch
    w = synth.RL_UPDATE
    H, D, T, B, M = w.heads, w.head_dim, w.tokens_per_frame, w.batch, w.chunk_tokens
    cache = A.astro_kvcache_create(B, H, D, T, w.sink_frames, w.window_frames, device=dev)
    A.astro_kvcache_append(cache, _rnd(dev, 10, (B, w.ctx_tokens, H, D)), _rnd(dev, 11, (B, w.ctx_tokens, H, D)), w.held_frames)
    q, kc, vc, do = (_rnd(dev, i, (B, M, H, D)) for i in range(4))
    o = torch.empty_like(q); lse = torch.empty((B, H, M), dtype=torch.float32, device=dev)
    dq, dk, dv = (torch.empty_like(q) for _ in range(3))
    ws = torch.empty(A.astro_chunk_attn_bwd_workspace_bytes(B, H, M, D), dtype=torch.uint8, device=dev)
    fwd = lambda: A.astro_chunk_attn_fwd(cache, q, kc, vc, w.scale, o=o, lse=lse)
    bwd = lambda: A.astro_chunk_attn_bwd(cache, q, kc, vc, o, lse, do, w.scale, dq=dq, dk_chunk=dk, dv_chunk=dv,
                                         workspace=ws)
    for _ in range(3):
        fwd(); bwd()
    ms_f, ms_b = _event_ms(fwd, reps), _event_ms(bwd, reps)
    A.astro_last_device_status()
    tf = lambda fl, ms: fl / (ms * 1e-3) / 1e12
    total = tf(w.fwd_flops() + w.bwd_flops(), ms_f + ms_b)
    return {"workload": "rl_update", "metric": "chunk_attn_fwd_bwd_tflops", "unit": "TFLOP/s", "value": total,
            "fwd": {"ms": ms_f, "tflops": tf(w.fwd_flops(), ms_f)},
            "bwd": {"ms": ms_b, "tflops": tf(w.bwd_flops(), ms_b)},
            "config": "B=2 H=12 D=128, 4680 q/k with grads over 28080 detached keys; %d launches back to back" % reps,
            "frac_of_bf16_burst": total / peaks["bf16_burst"], "frac_of_bf16_sustained": total / peaks["bf16_sustained"]}


def measure_score_sensitivity(A, dev, peaks, reps=10):
    """Forward at the layer shape with the scores multiplied by 8 (scale 8/sqrt(D)): N(0,1) inputs then give peaky
    softmax rows instead of near-uniform ones, which is closer to post-norm Q K products of a trained model."""
    import torch
    w = synth.LAYER_FWD
    H, D, T, B, M = w.heads, w.head_dim, w.tokens_per_frame, w.batch, w.chunk_tokens
    cache = A.astro_kvcache_create(1, H, D, T, w.sink_frames, w.window_frames, device=dev)
    A.astro_kvcache_append(cache, _rnd(dev, 10, (1, w.ctx_tokens, H, D)), _rnd(dev, 11, (1, w.ctx_tokens, H, D)), w.held_frames)
    q, kc, vc = (_rnd(dev, i, (B, M, H, D)) for i in range(3))
    o = torch.empty_like(q); lse = torch.empty((B, H, M), dtype=torch.float32, device=dev)
    out = {"workload": "layer forward, scores x1 and x8", "kernel": "chunk_attn_fwd_kernel<128>"}
    for gain in (1, 8):
        fwd = lambda: A.astro_chunk_attn_fwd(cache, q, kc, vc, gain * w.scale, o=o, lse=lse)
        for _ in range(3):
            fwd()
        ms = _event_ms(fwd, reps)
        A.astro_last_device_status()
        out["x%d" % gain] = {"ms": ms, "tflops": w.fwd_flops() / (ms * 1e-3) / 1e12,
                             "frac_of_bf16_burst": w.fwd_flops() / (ms * 1e-3) / 1e12 / peaks["bf16_burst"]}
    out["slowdown_x8"] = out["x8"]["ms"] / out["x1"]["ms"]
    return out


def measure_pair_kernel(A, dev, peaks, reps=10):
    """Forward on shapes of the workloads through the single-CTA kernel and through the CTA-pair kernel (two query
    tiles per K/V tile, tcgen05 cta_group::2), one JSON-able row per shape."""
    import torch
    H, D, T = 12, 128, 1560
    shapes = (("layer, B=1 (37 query tiles per head)", 1, 1, 18, 4680), ("rollout, B=4 per-sample caches, 12 held", 4, 4, 12, 4680),
              ("group of 8 on one prefix", 8, 1, 18, 4680), ("group of 24 on one prefix", 24, 1, 18, 4680),
              ("rl_update forward, B=2", 2, 2, 18, 4680), ("per-frame chunk, B=4, 20 held", 4, 4, 20, 1560),
              ("B=8, 4608 queries (36 tiles per head)", 8, 8, 18, 4608))
    rows = []
    for name, B, Bc, held, M in shapes:
        cache = A.astro_kvcache_create(Bc, H, D, T, 3, held, device=dev)
        A.astro_kvcache_append(cache, _rnd(dev, 10, (Bc, held * T, H, D)), _rnd(dev, 11, (Bc, held * T, H, D)), held)
        q, kc, vc = (_rnd(dev, i, (B, M, H, D)) for i in range(3))
        o = torch.empty_like(q); lse = torch.empty((B, H, M), dtype=torch.float32, device=dev)
        flops = 4.0 * B * H * M * (held * T + M) * D
        row = {"shape": name, "batch": B, "cache_batch": Bc, "queries": M, "keys": held * T + M}
        fwd = lambda: A.astro_chunk_attn_fwd(cache, q, kc, vc, 1.0 / float(np.sqrt(D)), o=o, lse=lse)
        try:
            for label, mode in (("single_cta", A.FWD_MODE_NORMAL), ("cta_pair", A.FWD_MODE_PAIR)):
                A.astro_debug_forward_mode(mode)
                for _ in range(3):
                    fwd()
                ms = _event_ms(fwd, reps)
                row[label] = {"ms": ms, "tflops": flops / (ms * 1e-3) / 1e12}
        finally:
            A.astro_debug_forward_mode(A.FWD_MODE_NORMAL)
        A.astro_last_device_status()
        row["pair_needed_safe_pass"] = A.astro_debug_pair_flag()
        row["pair_over_single_speed"] = row["single_cta"]["ms"] / row["cta_pair"]["ms"]
        rows.append(row)
        del cache, q, kc, vc, o, lse
        torch.cuda.empty_cache()
    return rows


def measure_variants(A, dev, peaks, reps=20):
    """Window presets of Tab. S1 (S = 3; 21 or 15 frames attended in total, the chunk included) with 3-frame and
    with per-frame chunks: forward of one layer, batch 4."""
    import torch
    H, D, T, Bv = 12, 128, 1560, 4
    rows = []
    for total, cf in ((21, 3), (21, 1), (15, 3), (15, 1)):
        held, Mv = total - cf, cf * T
        cache = A.astro_kvcache_create(Bv, H, D, T, 3, total - 3, device=dev)
        A.astro_kvcache_append(cache, _rnd(dev, 40, (Bv, held * T, H, D)), _rnd(dev, 41, (Bv, held * T, H, D)), held)
        qv, kv, vv = (_rnd(dev, 42 + i, (Bv, Mv, H, D)) for i in range(3))
        ov = torch.empty_like(qv); lv = torch.empty((Bv, H, Mv), dtype=torch.float32, device=dev)
        sc = 1.0 / float(np.sqrt(D))
        fwd = lambda: A.astro_chunk_attn_fwd(cache, qv, kv, vv, sc, o=ov, lse=lv)
        for _ in range(3):
            fwd()
        ms = _event_ms(fwd, reps)
        A.astro_last_device_status()
        flops = 4.0 * Bv * H * Mv * (held * T + Mv) * D
        rows.append({"attended_frames": total, "chunk_frames": cf, "batch": Bv, "queries": Mv, "keys": held * T + Mv,
                     "ms": ms, "tflops": flops / (ms * 1e-3) / 1e12,
                     "latent_frames_per_s_4_steps": Bv * cf / (4 * ms * 1e-3),
                     "frac_of_bf16_burst": flops / (ms * 1e-3) / 1e12 / peaks["bf16_burst"]})
        del cache
    return rows


def run_extra(args):
    """Rollout, clip-window update and context sweep on one GPU (device-resident inputs, CUDA events)."""
    import torch
    from paper_2603_17051_b200 import binding as A
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peaks = measured_peaks()

    def rnd(i, shape):
        bits = synth.normal_bf16(synth.tensor_seed(9, i), shape)
        return torch.from_numpy(bits.view(np.int16)).to(dev).view(torch.bfloat16)

    H, D, T, c = 12, 128, 1560, 3
    M = c * T
    if args.workload == "rollout":
        print(json.dumps(measure_rollout(A, dev, peaks, chunks=80, reading=args.reading)))
        return 0
    if args.workload == "variants":
        for row in measure_variants(A, dev, peaks):
            print(json.dumps(dict(workload="variants", **row)))
        return 0
    if args.workload == "pair":
        for row in measure_pair_kernel(A, dev, peaks):
            print(json.dumps(dict(workload="pair", **row)))
        return 0
    if args.workload == "sensitivity":
        print(json.dumps(measure_score_sensitivity(A, dev, peaks)))
        return 0
    if args.workload == "nft":
        # policy loss + selective KL + gradient on the velocity tensors of a 3-frame window (16 x 60 x 104 latents)
        Bn, E = 96, 3 * 16 * 60 * 104
        vt, vo, vr, tg = (rnd(30 + i, (Bn, E)) for i in range(4))
        r = torch.rand(Bn, device=dev); wp = torch.full((Bn,), 1.0 / (Bn * E), device=dev)
        wk = torch.full((Bn,), 1e-4 / E, device=dev)
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
        outs = (torch.empty(Bn, device=dev), torch.empty(Bn, device=dev), torch.empty_like(vt))
        call = lambda: A.astro_nft_loss(vt, vo, vr, tg, r, 1.0, w_policy=wp, w_kl=wk, out=outs)
        for _ in range(3):
            call()
        # 288 MB touched per call (larger than L2); 20 calls back to back so that the device, not the host
        # submitting two memsets and a kernel per call, sets the pace
        ms = _event_ms(call, 20)
        byts = 5 * 2 * Bn * E
        print(json.dumps({"workload": "nft", "metric": "nft_loss_hbm_gbs", "value": byts / ms / 1e6, "unit": "GB/s",
                          "ms": ms, "bytes_moved": byts, "config": "96 samples x 299520 elements, 4 bf16 reads + 1 bf16 write, 20 calls back to back",
                          "roofline": {"bound": "hbm", "achieved": byts / ms / 1e6, "peak": peaks["hbm"], "unit": "GB/s",
                                       "frac": byts / ms / 1e6 / peaks["hbm"]}}))
        return 0
    if args.workload == "group":
        # clip-level group-wise sampling: G candidate chunks decode against one frozen, shared prefix
        w = synth.LAYER_FWD
        G = args.group
        Bc = G if args.replicated else 1
        cache = A.astro_kvcache_create(Bc, H, D, T, w.sink_frames, w.window_frames, device=dev)
        kx, vx = rnd(10, (1, w.ctx_tokens, H, D)), rnd(11, (1, w.ctx_tokens, H, D))
        if args.replicated:
            kx, vx = kx.expand(G, -1, -1, -1).contiguous(), vx.expand(G, -1, -1, -1).contiguous()
        A.astro_kvcache_append(cache, kx, vx, w.held_frames)
        del kx, vx
        q, kc, vc = (rnd(i, (G, M, H, D)) for i in range(3))
        o = torch.empty_like(q); lse = torch.empty((G, H, M), dtype=torch.float32, device=dev)
        fwd = lambda: A.astro_chunk_attn_fwd(cache, q, kc, vc, w.scale, o=o, lse=lse)
        for _ in range(3):
            fwd()
        ms = _event_ms(fwd, args.steps if args.steps < 50 else 10)
        A.astro_last_device_status()
        flops = G * w.fwd_flops()
        print(json.dumps({"workload": "group", "G": G, "prefix": "replicated" if args.replicated else "shared",
                          "metric": "chunk_attn_fwd_tflops", "value": flops / (ms * 1e-3) / 1e12, "unit": "TFLOP/s",
                          "ms": ms, "cache_bytes": 2 * Bc * H * (w.sink_frames + w.window_frames) * T * D * 2,
                          "config": "G x (4680 q, 12 heads, D=128) over 28080 cached + 4680 chunk keys",
                          "frac_of_bf16_sustained": flops / (ms * 1e-3) / 1e12 / peaks["bf16_sustained"]}))
        return 0
    if args.workload == "rl_update":
        print(json.dumps(measure_rl_update(A, dev, peaks)))
        return 0
    # sweep: 30 independent layers x 8 samples x 7 chunks x 4 denoising steps, keys per query held fixed
    B, layers, chunks, steps = 8, 30, 7, 4
    q, kc, vc = (rnd(i, (B, M, H, D)) for i in range(3))
    o = torch.empty_like(q); lse = torch.empty((B, H, M), dtype=torch.float32, device=dev)
    scale = 1.0 / float(np.sqrt(D))
    for n_k in synth.SWEEP_KEYS:
        n_ctx = max(n_k - M, 0)
        n_kc = min(n_k, M)
        caches = []
        if n_ctx:
            tpf = 780                                          # half frames, so 16380 keys (10.5 frames) fit exactly
            frames = n_ctx // tpf
            per_cache = 2 * B * H * n_ctx * D * 2
            n_alloc = layers if per_cache * layers < 120e9 else 1
            fill_k, fill_v = rnd(20, (B, n_ctx, H, D)), rnd(21, (B, n_ctx, H, D))
            for _ in range(n_alloc):
                cch = A.astro_kvcache_create(B, H, D, tpf, 0, frames, device=dev)
                A.astro_kvcache_append(cch, fill_k, fill_v, frames)
                caches.append(cch)
            del fill_k, fill_v
        kcs, vcs = kc[:, :n_kc].contiguous(), vc[:, :n_kc].contiguous()

        def sweep_pass():
            for _ in range(chunks):
                for _ in range(steps):
                    for layer in range(layers):
                        cch = caches[layer % len(caches)] if caches else None
                        A.astro_chunk_attn_fwd(cch, q, kcs, vcs, scale, o=o, lse=lse)
        for layer in range(min(layers, 3)):
            A.astro_chunk_attn_fwd(caches[layer % len(caches)] if caches else None, q, kcs, vcs, scale, o=o, lse=lse)
        ms = _event_ms(sweep_pass, 1)
        A.astro_last_device_status()
        flops = 4.0 * B * H * M * (n_ctx + n_kc) * D * layers * chunks * steps
        print(json.dumps({"workload": "sweep", "keys": n_k, "metric": "rollout_latent_frames_per_s",
                          "value": chunks * c * B / (ms * 1e-3), "unit": "latent-frames/s (all 8 samples)",
                          "per_sample_latent_frames_per_s": chunks * c / (ms * 1e-3), "ms_total": ms,
                          "tflops": flops / (ms * 1e-3) / 1e12,
                          "frac_of_bf16_sustained": flops / (ms * 1e-3) / 1e12 / peaks["bf16_sustained"],
                          "caches_resident": len(caches), "note": "attention only; 30 layers x 7 chunks x 4 steps"}))
        del caches
        torch.cuda.empty_cache()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", choices=("ours", "reference"), default="ours")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--dry-run", action="store_true",
                    help="check the launch path only: no GPU work, made-up step time, gloo rendezvous")
    ap.add_argument("--no-legs", action="store_true", help="layer workload: skip the rollout / rl_update / variant sub-records")
    ap.add_argument("--rollout-chunks", type=int, default=16,
                    help="chunks of the rollout sub-record of the default line (the full workload has 80)")
    ap.add_argument("--workload", choices=("layer", "rollout", "rl_update", "sweep", "group", "nft", "variants", "sensitivity", "pair"), default="layer",
                    help="layer (default): the contract line; the others print one JSON line per extra workload")
    ap.add_argument("--group", type=int, default=24, help="group workload: candidates G decoding against one prefix")
    ap.add_argument("--replicated", action="store_true",
                    help="group workload: give every candidate its own copy of the prefix (comparison)")
    ap.add_argument("--reading", choices=("A", "B"), default="A",
                    help="rollout only: A = window capacity counts the chunk (12 held + chunk), B = 15 held + chunk")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours" and args.workload == "layer":
        return relaunch_under_torchrun(args, sys.argv[1:])
    if args.impl == "reference":
        return run_reference(args)
    if args.dry_run:
        return run_dry(args)
    if args.workload != "layer":
        return run_extra(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
