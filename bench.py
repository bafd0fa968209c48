#!/usr/bin/env python
"""Benchmark of the KSA attention forward hot path on B200.

A "step" is one pass of the whole hot path (pack -> summary-row kernel -> text-row
tensor-core kernel) over one batch of synthetic input shaped like the paper's 128K
long-context workload (131,072 text tokens, chunk size 8 with one summary token, 128
sliding chunks, GQA 32/4, head dim 128, bf16).  The metric is visible TFLOP/s: only the
(query, key) pairs the KSA mask makes visible count, 4*D flops each per query head.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 128k] [--layout P]
    python bench.py --impl reference ...      # the CPU oracle on a bounded row sample

N > 1 (under torchrun): every rank runs its own independent batch (weak scaling, no
data-path collective); the value is the aggregate over ranks, timed as max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2604_24432_b200 import dist_utils, synth

METRIC = "KSA attn fwd visible TFLOP/s & text tok/s at 128K, % of B200 BF16 peak"

TRAFFIC_RECORDS = os.path.join(ROOT, "profiles", "ncu_dram_traffic.json")


def ncu_traffic(kernel: str, workload: str, layout: str):
    """DRAM bytes (read + write) per launch of `kernel` from the ncu capture recorded in profiles/ncu_dram_traffic.json,
    or None: no record for this kernel and workload, or the kernel's source file has changed since the counters were
    taken (the record carries the file's SHA-256)."""
    import hashlib
    try:
        with open(TRAFFIC_RECORDS) as f:
            records = json.load(f)["records"]
    except (OSError, ValueError, KeyError):
        return None
    for r in records:
        if r.get("kernel") == kernel and r.get("workload") == workload and r.get("layout") == layout:
            try:
                with open(os.path.join(ROOT, r["source"]), "rb") as f:
                    if hashlib.sha256(f.read()).hexdigest() != r["source_sha256"]:
                        return None
            except OSError:
                return None
            return float(r["dram_bytes_per_launch"])
    return None


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return dict(source="measured", hbm_gbs=float(d["hbm_gbs"]), bf16_burst=float(d["bf16_tflops"]),
                    bf16_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])))
    return dict(source="fallback", hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0)


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    REASONS = {
        0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
        0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
        0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting",
    }

    def __init__(self, index: int, period: float = 0.05):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self.period = period
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _run(self):
        while not self._stop.is_set():
            try:
                self.samples.append(int(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM)))
                mask = int(self.nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["nvml_unavailable"]}
        reasons = sorted(self.reasons - {"gpu_idle"})
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz, "reasons": reasons}


def spawn_ranks(n: int) -> int:
    """`python bench.py --gpus N` outside torchrun: build once, then start N ranks of this very command under
    torch.distributed.run on this node (one process per GPU) and pass their output through."""
    import socket
    import subprocess
    if not os.environ.get("KSA_BENCH_LAUNCH_TEST"):
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
        have = torch.cuda.device_count()
        if n > have:
            raise SystemExit(f"bench.py --gpus {n}: this node has {have} GPU(s)")
        from paper_2604_24432_b200 import build as ksa_build
        ksa_build.build()
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    env = dict(os.environ, KSA_BENCH_BUILT="1")
    return subprocess.call(cmd, env=env)


def run_launch_test(args):
    """KSA_BENCH_LAUNCH_TEST=1 (the CPU test of the launcher): the ranks that spawn_ranks started meet over gloo, time a
    stand-in step (no kernel, no attention arithmetic), reduce the time with MAX over ranks and rank 0 prints the line's
    launch-related keys.  Nothing here measures anything."""
    import torch.distributed as dist
    rank, world, _ = dist_env()
    dist.init_process_group("gloo")
    dist.barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        time.sleep(0.001 * (rank + 1))                  # the slower rank must set the time
    ms = dist_utils.max_over_ranks(1e3 * (time.perf_counter() - t0) / args.steps)
    dist.barrier()
    if rank == 0:
        print(json.dumps({"launch_test": True, "n_gpus": world, "steps": args.steps, "ms_per_step": ms,
                          "built_by_launcher": bool(os.environ.get("KSA_BENCH_BUILT"))}))
    dist.destroy_process_group()
    return 0


def build_once(rank: int, world: int):
    """One build per node: the launcher has built already, or rank 0 builds while the others wait at a barrier
    (the process group must exist when world > 1)."""
    from paper_2604_24432_b200 import build as ksa_build
    if world == 1:
        ksa_build.build()
        return
    import torch.distributed as dist
    if rank == 0 and not os.environ.get("KSA_BENCH_BUILT"):
        ksa_build.build()
    dist.barrier()


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def workload_and_layout(args):
    wl = synth.WORKLOADS[args.workload]
    layout = {"P": synth.LAYOUT_P, "G": synth.LAYOUT_G, "F": synth.LAYOUT_F}[args.layout]
    return wl, layout


def base_config(wl, layout, world):
    return {
        "workload": f"{wl.name} ({wl.note})", "layout": f"{layout.name}: k={layout.k} m={layout.m} C={layout.C}",
        "text_tokens_per_gpu": int(sum(wl.text_lens)), "heads": f"{wl.Hq}q/{wl.Hkv}kv", "head_dim": wl.D,
        "l2_policy": "inputs larger than L2 (no flush)", "parallelism": f"replicas x{world}" if world > 1 else "1 GPU",
    }


# ---------------------------------------------------------------------------------------
# reference arm: the CPU oracle, as it stands, on a bounded sample of rows per step
# ---------------------------------------------------------------------------------------
def oracle_sample_rows(wl, layout, n_rows, seed):
    from oracle import ksa_oracle as orc
    total = sum(orc.aug_len(n, layout.k, layout.m) for n in wl.text_lens)
    rng = np.random.default_rng(seed)
    return np.sort(rng.choice(total, size=min(n_rows, total), replace=False)).astype(np.int64), total


def time_oracle(wl, layout, q, k, v, rows):
    from oracle import ksa_oracle as orc
    t0 = time.perf_counter()
    _, _, cnt = orc.fwd(synth.bits(q), synth.bits(k), synth.bits(v), wl.text_lens, layout.k, layout.m,
                        layout.C, wl.scale, rows=rows)
    dt = time.perf_counter() - t0
    flops = 4.0 * wl.D * wl.Hq * float(cnt.sum())
    return dt, flops, orc.num_threads()


def run_reference(args):
    rank, world, _ = dist_env()
    if rank != 0:
        return 0
    wl, layout = workload_and_layout(args)
    # a bounded sample per step, sized so that warm-up plus timed steps stay within a few minutes of host time
    # (about 9,000 rows in all, at most --oracle-rows per step)
    per_step = max(32, min(args.oracle_rows, 9000 // max(1, args.warmup + args.steps)))
    rows, total = oracle_sample_rows(wl, layout, per_step, 1234)
    q, k, v = synth.make_qkv(wl, total)
    times, flops = [], 0.0
    cores = 0
    for it in range(args.warmup + args.steps):
        dt, flops, cores = time_oracle(wl, layout, q, k, v, rows)
        if it >= args.warmup:
            times.append(dt)
    ms = 1e3 * sum(times) / len(times)
    value = flops / (ms * 1e-3) / 1e12
    sample = f"{len(rows)} random augmented rows of the workload per step, all {wl.Hq} heads"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic (seeded, bf16 inputs)",
        "config": base_config(wl, layout, 1),
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))
    return 0


# ---------------------------------------------------------------------------------------
# our arm
# ---------------------------------------------------------------------------------------
def run_ours(args):
    from paper_2604_24432_b200 import binding as ksa
    from paper_2604_24432_b200 import build as ksa_build

    rank, world, local = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    build_once(rank, world)
    wl, layout = workload_and_layout(args)
    if world > 1:   # independent batch per rank
        wl = dist_utils.rank_workload(wl, rank)
    kflags = {"auto": 0, "single": ksa.KSA_FLAG_SINGLE_CTA_KERNEL, "pair": ksa.KSA_FLAG_CTA_PAIR_KERNEL}[args.text_kernel]
    prob = ksa.Problem(wl.text_lens, layout.k, layout.m, layout.C, wl.Hq, wl.Hkv, wl.D, wl.scale, kflags)
    total = ksa.total_aug_len(prob)
    pairs = ksa.visible_pairs(prob)
    flops = 4.0 * wl.D * wl.Hq * pairs
    n_text = int(sum(wl.text_lens))

    qh, kh, vh = synth.make_qkv(wl, total, pin=True)
    q, k, v = qh.to(dev), kh.to(dev), vh.to(dev)
    out = torch.empty((total, wl.Hq, wl.D), dtype=torch.bfloat16, device=dev)
    lse = torch.empty((wl.Hq, total), dtype=torch.float32, device=dev)
    ws = torch.empty(ksa.workspace_bytes(prob), dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream(dev)
    # ---- cold call: a fresh context builds and uploads the schedule inside the call ------------
    cold_ctx = ksa.Context(local)
    cold_ctx.attn_fwd(prob, q, k, v, out, lse, ws)       # kernel set-up (shared-memory opt-in) of this process
    torch.cuda.synchronize()
    cold_ctx.close()
    ctx = ksa.Context(local)
    t_cold = time.perf_counter()
    ctx.attn_fwd(prob, q, k, v, out, lse, ws)
    torch.cuda.synchronize()
    cold_ms = 1e3 * (time.perf_counter() - t_cold)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing -------------------------------------------------------
    for _ in range(max(args.warmup, 3)):
        ctx.attn_fwd(prob, q, k, v, out, lse, ws)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0, "device-side wait gave up"
    ctx.enable_kernel_timing(True)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    text_ms = []
    launches0 = ctx.launch_count()
    barrier()
    with ClockSampler(local) as clocks:
        ev[0].record(stream)
        for i in range(args.steps):
            ctx.attn_fwd(prob, q, k, v, out, lse, ws)
            ev[i + 1].record(stream)
            # the library's own event pair brackets the text-row kernel of this step
            text_ms.append(ctx.text_kernel_ms())
        barrier()
    launches = ctx.launch_count() - launches0
    total_ms = ev[0].elapsed_time(ev[args.steps])
    step_ms = [ev[i].elapsed_time(ev[i + 1]) for i in range(args.steps)]
    ctx.enable_kernel_timing(False)
    assert ctx.device_status() == 0, "device-side wait gave up"
    total_ms = dist_utils.max_over_ranks(total_ms, dev)
    ms_per_step = total_ms / args.steps
    value = dist_utils.aggregate_rate(flops, world, ms_per_step) / 1e12
    tok_s = dist_utils.aggregate_rate(n_text, world, ms_per_step)

    # ---- end to end through the host entry point ----------------------------------------
    e2e = None
    if not args.no_e2e:
        out_h = torch.empty((total, wl.Hq, wl.D), dtype=torch.bfloat16).pin_memory()
        lse_h = torch.empty((wl.Hq, total), dtype=torch.float32).pin_memory()
        del out, lse, ws
        staging = torch.empty(ksa.host_staging_bytes(prob), dtype=torch.uint8, device=dev)
        ctx.attn_fwd_host(prob, qh, kh, vh, out_h, lse_h, staging)       # warm-up
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.e2e_steps):
            ctx.attn_fwd_host(prob, qh, kh, vh, out_h, lse_h, staging)
        e1.record(stream)
        barrier()
        e2e_ms = e0.elapsed_time(e1) / args.e2e_steps
        e2e_ms = dist_utils.max_over_ranks(e2e_ms, dev)
        h2d = qh.numel() * 2 + kh.numel() * 2 + vh.numel() * 2
        d2h = out_h.numel() * 2 + lse_h.numel() * 4
        # the box's pinned-memory copy rates, measured here: the floor of the end-to-end time is the slower of the two
        # directions (they overlap) -- the compute hides behind them
        def copy_gbs(dst, src, reps=3):
            torch.cuda.synchronize()
            c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            c0.record(stream)
            for _ in range(reps):
                dst.copy_(src, non_blocking=True)
            c1.record(stream)
            torch.cuda.synchronize()
            return reps * src.numel() * src.element_size() / (c0.elapsed_time(c1) * 1e-3) / 1e9
        dq = torch.empty_like(q)
        h2d_gbs = copy_gbs(dq, qh)
        d2h_gbs = copy_gbs(out_h, dq)
        del dq
        floor_ms = 1e3 * max(h2d / (h2d_gbs * 1e9), d2h / (d2h_gbs * 1e9))
        e2e = {"value": world * flops / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s", "ms_per_step": e2e_ms,
               "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": args.e2e_steps,
               "api": "ksa_attn_fwd_host (pinned host tensors)",
               "pcie": {"h2d_gbs": h2d_gbs, "d2h_gbs": d2h_gbs, "floor_ms": floor_ms,
                        "note": "floor = the slower direction's bytes / its measured pinned copy rate (the two directions and the compute overlap)",
                        "frac_of_floor": floor_ms / e2e_ms}}

    if rank != 0:
        return 0

    # ---- roofline of the dominant kernel (text rows, tensor-bound) ------------------------
    peaks = load_peaks()
    text_pairs = pairs - summary_pairs(wl, layout)
    text_flops = 4.0 * wl.D * wl.Hq * text_pairs
    text_avg_ms = sum(text_ms) / len(text_ms)
    achieved = text_flops / (text_avg_ms * 1e-3) / 1e12
    kernel_name = "ksa_text_pair_kernel" if args.text_kernel == "pair" else "ksa_text_tc_kernel"
    traffic = ncu_traffic(kernel_name, wl.name, layout.name)
    roofline = {
        "bound": "tensor", "achieved": achieved, "peak": peaks["bf16_burst"], "unit": "TFLOP/s",
        "frac": achieved / peaks["bf16_burst"], "traffic": traffic,
        "peak_source": f"of {peaks['source']} (burst bf16 GEMM rate: the dense BF16 tensor rate this box attains)",
        "frac_of_sustained_peak": achieved / peaks["bf16_sustained"], "sustained_peak": peaks["bf16_sustained"],
        "frac_of_nominal_2250": achieved / 2250.0,
        "kernel": kernel_name, "kernel_ms_avg": text_avg_ms, "kernel_ms_median": statistics.median(text_ms),
        "kernel_ms_min": min(text_ms), "kernel_share_of_step": text_avg_ms / ms_per_step,
    }

    # ---- CPU baseline: the oracle on a bounded sample (rank 0, N = 1 only) -----------------
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        rows, _ = oracle_sample_rows(wl, layout, args.oracle_rows, 1234)
        dt, oflops, cores = time_oracle(wl, layout, qh, kh, vh, rows)
        cpu = {"value": oflops / dt / 1e12, "unit": "TFLOP/s", "cores": cores, "kind": "oracle",
               "sample": f"{len(rows)} random augmented rows, all {wl.Hq} heads, {dt:.1f} s"}

    line = {
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "ms_per_step_median": statistics.median(step_ms),
        "ms_per_step_min": min(step_ms), "cold_call_ms": cold_ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic (seeded)",
        "config": base_config(wl, layout, world),
        "text_tok_per_s": tok_s, "visible_tflop_per_step": flops / 1e12,
        "pct_of_peak": {"measured_burst": 100 * value / world / peaks["bf16_burst"],
                        "measured_sustained": 100 * value / world / peaks["bf16_sustained"],
                        "nominal_2250": 100 * value / world / 2250.0, "source": peaks["source"]},
        "clocks": clocks.summary(), "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline,
        "cpu_baseline": cpu,
    }
    print(json.dumps(line))
    return 0


# ---------------------------------------------------------------------------------------
# decode path (secondary line): one auto-regressive step over the Summary KV cache
# ---------------------------------------------------------------------------------------
def run_decode(args):
    """python bench.py --decode: B sequences at a 128K-token context (layout P, GQA 32/4, D 128), each step
    appends one text token per sequence and attends over the cache slice; every k-th step is followed by
    the chunk's summary step.  HBM-bound: the roofline is the measured copy bandwidth."""
    from paper_2604_24432_b200 import binding as ksa
    from paper_2604_24432_b200 import build as ksa_build
    rank, world, local = dist_env()
    if rank != 0:
        return 0
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    ksa_build.build()
    Hq, Hkv = (int(x) for x in args.decode_heads.split("/"))
    B, k, C, D = args.decode_batch, 8, 128, 128
    ctx_len = 131072
    steps, warm = args.steps, max(args.warmup, 3)
    spec = ksa.CacheSpec(B, k, C, ctx_len // k + (steps + warm) // k + 2, Hq, Hkv, D, float(np.float32(1.0 / np.sqrt(D))))
    ctx = ksa.Context(local)
    cache = ksa.DecodeCache(ctx, spec)
    g = torch.Generator(device=dev).manual_seed(5)
    cache.kcache.normal_(generator=g); cache.vcache.normal_(generator=g)
    pos0 = ctx_len - k * ((warm + k - 1) // k)          # chunk-aligned start so that the timed region starts at ctx_len
    cache.state[:, 0] = pos0; cache.state[:, 1] = pos0 // k
    q = torch.randn((B, Hq, D), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
    kn = torch.randn((B, Hkv, D), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
    vn = torch.randn((B, Hkv, D), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
    out = torch.empty((B, Hq, D), dtype=torch.bfloat16, device=dev)
    lse = torch.empty((B, Hq), dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream(dev)

    def step(pos):
        cache.decode_text(q, kn, vn, out, lse)
        if (pos + 1) % k == 0:
            cache.decode_summary(q, kn, vn, out, lse)
        return pos + 1

    pos = pos0
    while pos < ctx_len:
        pos = step(pos)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    steps = max(k, (steps // k) * k)            # whole chunks: k text steps and the chunk's summary step
    launches0 = ctx.launch_count()
    bytes_read = 0
    for i in range(steps):
        lo, hi = ksa.cache_slice(spec, pos + i, False)
        bytes_read += B * Hkv * (hi - lo) * D * 2 * 2
        if (pos + i + 1) % k == 0:
            bytes_read += B * Hkv * (k + 1) * D * 2 * 2
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    graph = None
    if not args.no_graph:
        # the step kernels take everything that changes from the device-side state, so one chunk's worth
        # of steps is captured once and replayed (no launch gaps between the four kernels of a step)
        launches_per_chunk = ctx.launch_count()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            p_ = pos
            for _ in range(k):
                p_ = step(p_)
        launches_per_chunk = ctx.launch_count() - launches_per_chunk
        stream = torch.cuda.current_stream(dev)
    with ClockSampler(local) as clocks:
        e0.record(stream)
        if graph is not None:
            for _ in range(steps // k):
                graph.replay()
            pos += steps
        else:
            for _ in range(steps):
                pos = step(pos)
        e1.record(stream)
        torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    assert ctx.device_status() == 0
    st = cache.state.cpu().numpy()
    assert (st[:, 0] == pos).all() and (st[:, 1] == pos // k).all()
    peaks = load_peaks()
    gbs = bytes_read / steps / (ms * 1e-3) / 1e9
    cache_gb = 2 * cache.kcache.numel() * 2 / 1e9
    line = {
        "metric": "KSA decode step over the Summary KV cache: tokens/s at a 128K context", "value": B / (ms * 1e-3), "unit": "tokens/s",
        "n_gpus": 1, "steps": steps, "warmup": warm, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic (seeded)",
        "config": {"workload": f"decode, {B} sequences at {ctx_len} cached text tokens each", "layout": f"P: k={k} m=1 C={C}",
                   "heads": f"{Hq}q/{Hkv}kv", "head_dim": D, "cache_gb": cache_gb,
                   "l2_policy": "the cache slices read per step are larger than L2 (no flush)", "parallelism": "1 GPU",
                   "launch": "CUDA graph of one chunk (k text steps + its summary step), replayed" if graph is not None else "plain launches"},
        "clocks": clocks.summary(),
        "gpu_launches": int(launches_per_chunk * (steps // k)) if graph is not None else int(ctx.launch_count() - launches0),
        "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
                     # dram__bytes_read.sum + dram__bytes_write.sum of one ksa_decode_attn_kernel launch (ncu; see profiles/),
                     # for the default batch of 32 sequences at a 128K context
                     "traffic": 1.137e9 if (B, ctx_len) == (32, 131072) else None,
                     "peak_source": f"of {peaks['source']} (copy bandwidth)",
                     "kernel": "ksa_decode_attn_kernel (+ append, merge, commit)",
                     "bytes_per_step": bytes_read / steps},
        "e2e": None, "cpu_baseline": None,
    }
    print(json.dumps(line))
    return 0


# ---------------------------------------------------------------------------------------
# backward pass (secondary line)
# ---------------------------------------------------------------------------------------
def run_backward(args):
    """python bench.py --backward [--workload 32k]: forward once, then the backward pass timed.  Visible FLOPs of
    the backward pass = 2.5 x the forward's (five products of the same visible pairs instead of two)."""
    from paper_2604_24432_b200 import binding as ksa
    from paper_2604_24432_b200 import build as ksa_build
    rank, world, local = dist_env()
    if rank != 0:
        return 0
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    ksa_build.build()
    wl, layout = workload_and_layout(args)
    prob = ksa.Problem(wl.text_lens, layout.k, layout.m, layout.C, wl.Hq, wl.Hkv, wl.D, wl.scale)
    total = ksa.total_aug_len(prob)
    flops = 2.5 * 4.0 * wl.D * wl.Hq * ksa.visible_pairs(prob)
    qh, kh, vh = synth.make_qkv(wl, total)
    q, k, v = qh.to(dev), kh.to(dev), vh.to(dev)
    del qh, kh, vh
    g = torch.Generator(device=dev).manual_seed(9)
    dout = torch.randn((total, wl.Hq, wl.D), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
    out = torch.empty_like(q); lse = torch.empty((wl.Hq, total), dtype=torch.float32, device=dev)
    ws = torch.empty(max(256, ksa.workspace_bytes(prob)), dtype=torch.uint8, device=dev)
    ctx = ksa.Context(local)
    ctx.attn_fwd(prob, q, k, v, out, lse, ws)
    del ws
    dq = torch.empty_like(q); dk = torch.empty_like(k); dv = torch.empty_like(v)
    wsb = torch.empty(ksa.bwd_workspace_bytes(prob), dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream(dev)
    for _ in range(max(args.warmup, 3)):
        ctx.attn_bwd(prob, q, k, v, out, lse, dout, dq, dk, dv, wsb)
    torch.cuda.synchronize()
    launches0 = ctx.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local) as clocks:
        e0.record(stream)
        for _ in range(args.steps):
            ctx.attn_bwd(prob, q, k, v, out, lse, dout, dq, dk, dv, wsb)
        e1.record(stream)
        torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    assert ctx.device_status() == 0
    peaks = load_peaks()
    val = flops / (ms * 1e-3) / 1e12
    line = {
        "metric": "KSA attn bwd visible TFLOP/s (2.5 x forward FLOPs)", "value": val, "unit": "TFLOP/s", "n_gpus": 1,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic (seeded)", "config": base_config(wl, layout, 1),
        "clocks": clocks.summary(), "gpu_launches": int(ctx.launch_count() - launches0),
        "roofline": {"bound": "tensor", "achieved": val, "peak": peaks["bf16_sustained"], "unit": "TFLOP/s",
                     "frac": val / peaks["bf16_sustained"], "traffic": None,
                     "peak_source": f"of {peaks['source']} (sustained bf16 GEMM)", "kernel": "ksa_bwd_dq_tc_kernel + ksa_bwd_dkv_tc_kernel (tcgen05; whole step incl. pack, prep, summary rows, finish)"},
        "e2e": None, "cpu_baseline": None,
    }
    print(json.dumps(line))
    return 0


# dram__bytes_read.sum + dram__bytes_write.sum of one ksa_prep_kernel launch (ncu; see profiles/)
NCU_PREP_KERNEL_DRAM_BYTES = {("128k", "P"): 3.160e9}


def run_seq_parallel(args):
    """Secondary line (--seq-parallel): ONE batch shared by all ranks.  Every rank owns a work-balanced part of the
    query rows (ksa_part_rows); a step is the exchange (all-gather of the ranks' rows of k and v over NCCL) plus the
    part's attention.  Total work is fixed as N grows: "scaling": "strong"."""
    from paper_2604_24432_b200 import binding as ksa
    from paper_2604_24432_b200 import build as ksa_build
    rank, world, local = dist_env()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    build_once(rank, world)
    wl, layout = workload_and_layout(args)
    prob = ksa.Problem(wl.text_lens, layout.k, layout.m, layout.C, wl.Hq, wl.Hkv, wl.D, wl.scale)
    total = ksa.total_aug_len(prob)
    flops = 4.0 * wl.D * wl.Hq * ksa.visible_pairs(prob)
    ctx = ksa.Context(local)
    ranges = [ctx.part_rows(prob, r, world) for r in range(world)]
    b, e = ranges[rank]
    qh, kh, vh = synth.make_qkv(wl, total)               # the same batch on every rank; a rank keeps its own rows only
    q = torch.zeros((total, wl.Hq, wl.D), dtype=torch.bfloat16, device=dev)
    q[b:e] = qh[b:e].to(dev)
    k_mine, v_mine = kh[b:e].to(dev), vh[b:e].to(dev)
    del qh, kh, vh
    out = torch.empty((total, wl.Hq, wl.D), dtype=torch.bfloat16, device=dev)
    lse = torch.empty((wl.Hq, total), dtype=torch.float32, device=dev)
    ws = torch.empty(max(256, ksa.workspace_bytes(prob)), dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream(dev)

    def step():
        if world > 1:
            k_full = dist_utils.all_gather_rows(k_mine, ranges, total)
            v_full = dist_utils.all_gather_rows(v_mine, ranges, total)
        else:
            k_full, v_full = k_mine, v_mine
        ctx.attn_fwd_part(prob, q, k_full, v_full, out, lse, ws, rank, world)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    launches0 = ctx.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local) as clocks:
        e0.record(stream)
        for _ in range(args.steps):
            step()
        e1.record(stream)
        barrier()
    assert ctx.device_status() == 0
    ms = dist_utils.max_over_ranks(e0.elapsed_time(e1), dev) / args.steps
    if rank == 0:
        peaks = load_peaks()
        val = flops / (ms * 1e-3) / 1e12
        cfg = base_config(wl, layout, 1)
        cfg["parallelism"] = f"sequence parallel x{world}: rows [{b}, {e}) of {total} on rank 0, all-gather of k and v per step"
        print(json.dumps({
            "metric": "KSA attn fwd visible TFLOP/s, one batch shared by all ranks", "value": val, "unit": "TFLOP/s",
            "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True,
            "scaling": "strong", "vs_baseline": None, "dtype": "bf16", "data": "synthetic (seeded)", "config": cfg,
            "clocks": clocks.summary(), "gpu_launches": int(ctx.launch_count() - launches0),
            "roofline": {"bound": "tensor", "achieved": val, "peak": world * peaks["bf16_sustained"], "unit": "TFLOP/s",
                         "frac": val / (world * peaks["bf16_sustained"]), "traffic": None,
                         "peak_source": f"of {peaks['source']} (sustained bf16 GEMM x {world})", "kernel": "ksa_text_tc_kernel (whole step incl. exchange)"},
            "e2e": None, "cpu_baseline": None}))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()
    return 0


def run_prep(args):
    """Secondary line: the Q/K/V preparation pass (position ids, interpolation at summary positions, rotary
    embedding) over the workload's q, k, v; HBM-bound, reported as algorithmic bytes per second."""
    from paper_2604_24432_b200 import binding as ksa
    from paper_2604_24432_b200 import build as ksa_build
    rank, world, local = dist_env()
    if rank != 0:
        return 0
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    ksa_build.build()
    wl, layout = workload_and_layout(args)
    prob = ksa.Problem(wl.text_lens, layout.k, layout.m, layout.C, wl.Hq, wl.Hkv, wl.D, wl.scale)
    total, S = ksa.total_aug_len(prob), ksa.total_summary_rows(prob)
    qh, kh, vh = synth.make_qkv(wl, total)
    q, k, v = qh.to(dev), kh.to(dev), vh.to(dev)
    del qh, kh, vh
    g = torch.Generator(device=dev).manual_seed(3)
    mk = lambda H: torch.randn((max(S, 1), H, wl.D), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
    qs, ks, vs = mk(wl.Hq), mk(wl.Hkv), mk(wl.Hkv)
    qo, ko, vo = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    ctx = ksa.Context(local)
    lam, theta = 0.5, 1.0e6                  # mid-way through the annealing window; Table 3's base after the 8K stage
    stream = torch.cuda.current_stream(dev)
    for _ in range(max(args.warmup, 3)):
        ctx.qkv_prepare(prob, q, k, v, qs, ks, vs, qo, ko, vo, lam, theta)
    torch.cuda.synchronize()
    launches0 = ctx.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local) as clocks:
        e0.record(stream)
        for _ in range(args.steps):
            ctx.qkv_prepare(prob, q, k, v, qs, ks, vs, qo, ko, vo, lam, theta)
        e1.record(stream)
        torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    row_bytes = (wl.Hq + 2 * wl.Hkv) * wl.D * 2
    alg_bytes = (2 * total + S) * row_bytes          # every row read and written once, summary projections read once
    peaks = load_peaks()
    gbs = alg_bytes / (ms * 1e-3) / 1e9
    line = {
        "metric": "KSA q/k/v preparation, augmented tokens/s", "value": total / (ms * 1e-3), "unit": "tokens/s", "n_gpus": 1,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic (seeded)", "config": base_config(wl, layout, 1),
        "clocks": clocks.summary(), "gpu_launches": int(ctx.launch_count() - launches0),
        "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
                     "traffic": NCU_PREP_KERNEL_DRAM_BYTES.get((wl.name, layout.name)),
                     "peak_source": f"of {peaks['source']} (copy bandwidth)", "kernel": "ksa_prep_kernel",
                     "algorithmic_bytes_per_launch": alg_bytes},
        "e2e": None, "cpu_baseline": None,
    }
    print(json.dumps(line))
    return 0


def summary_pairs(wl, layout):
    """Visible pairs of the summary rows (they run in their own small kernel)."""
    tot = 0
    for n in wl.text_lens:
        J = n // layout.k
        tot += J * sum(layout.k + r + 1 for r in range(layout.m))
    return tot


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="128k", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--layout", default="P", choices=["P", "G", "F"],
                    help="P, G: the paper's KSA layouts; F: full causal attention (the hybrid stack's full layers)")
    ap.add_argument("--text-kernel", default="auto", choices=["auto", "single", "pair"],
                    help="text-row kernel: the library's choice, the one-CTA kernel, or the CTA-pair kernel (cta_group::2)")
    ap.add_argument("--oracle-rows", type=int, default=3000)
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--decode", action="store_true", help="secondary line: the decode path over the Summary KV cache")
    ap.add_argument("--decode-batch", type=int, default=32)
    ap.add_argument("--decode-heads", default="32/4", help="decode: query heads / KV heads")
    ap.add_argument("--backward", action="store_true", help="secondary line: the backward pass")
    ap.add_argument("--seq-parallel", action="store_true",
                    help="secondary line: one batch shared by all ranks (work-balanced row parts, all-gather of k and v)")
    ap.add_argument("--prep", action="store_true", help="secondary line: the q/k/v preparation pass upstream of the attention")
    ap.add_argument("--no-graph", action="store_true", help="decode: plain launches instead of a replayed CUDA graph")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        return spawn_ranks(args.gpus)
    if "WORLD_SIZE" in os.environ and int(os.environ["WORLD_SIZE"]) != args.gpus:
        raise SystemExit(f"bench.py --gpus {args.gpus} under a launcher with WORLD_SIZE={os.environ['WORLD_SIZE']}")
    if os.environ.get("KSA_BENCH_LAUNCH_TEST"):
        return run_launch_test(args)
    if args.decode:
        return run_decode(args)
    if args.backward:
        return run_backward(args)
    if args.prep:
        return run_prep(args)
    if args.seq_parallel:
        return run_seq_parallel(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
