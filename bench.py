#!/usr/bin/env python
"""Benchmark of the cache-aware inference hot path: cached frames/s on B200.

A step is one pass of the whole path (matching, propagation, reuse copy, partial
convolutions, pooling, cache update) over one batch: one new frame for each of the
workload's independent video streams.  Default workload: "batched_stress" (32 streams of
1920x1080 video, VGG-16-shaped trunk at 224x224, bf16).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line (rank 0).  With --gpus N > 1 it must be started by torchrun; every
rank then runs its own set of streams (weak scaling, no collective on the data path) and
the timing is the maximum over ranks.
"""
from __future__ import annotations

import argparse
import ctypes
import json
import os
import statistics
import subprocess
import sys
import threading
import time
from concurrent.futures import ThreadPoolExecutor

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "cached_frames_per_sec"
UNIT = "frames/s"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=60)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=5)
    ap.add_argument("--streams", type=int, default=0, help="override the number of streams per GPU")
    ap.add_argument("--skip-k", type=int, default=1, help="Step 2 on every k-th block row / column only (Section 4); default 1 = all blocks")
    ap.add_argument("--search", default="", choices=["", "exhaustive", "diamond", "three_step"],
                    help="Step 2 search unit; default: the workload's (diamond)")
    ap.add_argument("--grouped", action="store_true", help="workload 3 with the cited AlexNet's two channel groups in layers 2, 4, 5")
    ap.add_argument("--cache-pool", action="store_true", help="also cache and reuse max-pooling outputs (Section 5's extension)")
    ap.add_argument("--per-block-regions", action="store_true", help="rectangles carry their blocks' own vectors (extension)")
    ap.add_argument("--no-lookahead", action="store_true", help="do not overlap the next frame's matching with this frame's inference")
    ap.add_argument("--matcher-only", action="store_true",
                    help="time Steps 1-5 alone (dc_cache_set_key + dc_match_blocks per step) and print a short JSON line; "
                         "a small, single-purpose run for profiling the matcher kernels")
    ap.add_argument("--reuse-copy", action="store_true",
                    help="time the reuse copy alone (Section 5 'Reuse', step 1) on one 64-channel 224x224 bf16 layer with "
                         "rectangles covering most of the map, through dc_conv_partial; prints a short JSON line")
    ap.add_argument("--conv-layer", default="",
                    help="CIN,COUT,HW[,K]: time one bf16 convolution layer alone (all tiles computed, --streams maps of HW x HW, K x K "
                         "kernel, default 3) through dc_conv_partial and print a short JSON line; DC_CONV_SCHEME selects the operand scheme")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    return ap.parse_args()


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"],
                    bf16_tflops_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from committed ncu captures.  Each entry names
# its capture and carries the SHA-256 of the kernel source it was taken with; when that source has changed since, the
# number no longer describes the kernels that run and null is printed instead.
CAPTURED_TRAFFIC = {
    "conv": {"bytes": 77.5e6, "source": "paper_1712_01670_b200/csrc/dc_conv_bf16.cu",
             "sha256": "966bb00e0613f45506f1a19eb309141c9cfb5bb83903a1be502c2d5ba1f571fc",
             "capture": "profiles/dram_traffic_batched_stress.md"},
    "matcher": {"bytes": 918.0e6, "source": "paper_1712_01670_b200/csrc/dc_match.cu",
                "sha256": "7430a21ee70e8b3abad717584591577772735c76ecba5750ad15af983c24b5b2",
                "capture": "profiles/dram_traffic_batched_stress.md"},
}


def captured_traffic(key, applies):
    import hashlib
    e = CAPTURED_TRAFFIC[key]
    if not applies or e["bytes"] is None:
        return None, None
    try:
        with open(os.path.join(ROOT, e["source"]), "rb") as f:
            sha = hashlib.sha256(f.read()).hexdigest()
    except OSError:
        return None, None
    if sha != e["sha256"]:
        return None, f"{e['capture']} predates the current {os.path.basename(e['source'])}"
    return e["bytes"], e["capture"]


def workload_config(w, n_streams, n_gpus):
    return {"workload": w.name, "streams_per_gpu": n_streams, "frame": f"{w.width}x{w.height}x3 uint8",
            "block": w.block, "range": w.range, "search": ("exhaustive", "diamond", "three_step")[w.search],
            "psnr_db": w.psnr_db, "expire_n": w.expire_n, "trunk_layers": len(w.layers),
            "parallelism": f"streams sharded over {n_gpus} GPU(s), no collective",
            "l2": "inputs larger than L2 (each step reads a fresh batch of frames)"}


def conv_flops_per_pixel(layers):
    return [2.0 * l["cout"] * l["cin"] * l["kh"] * l["kw"] if l["kind"] == 0 else 0.0 for l in layers]


# ---------------------------------------------------------------------------
# the oracle as CPU baseline / reference arm
# ---------------------------------------------------------------------------
def run_oracle_sample(w, n_frames, stream=0):
    """Times the oracle, as it stands, on frames 0..n_frames-1 of one stream.  Returns
    (frames/s, seconds, description)."""
    from oracle import deepcache_oracle as orc
    ws, bs = w.weights()
    quant = orc.QUANT_BF16 if w.dtype == 1 else orc.QUANT_NONE
    oc = orc.OracleCache(w.width, w.height, w.layers, ws, bs, block=w.block, search_range=w.range,
                         search_kind=w.search, psnr_db=w.psnr_db, expire_n=w.expire_n, quant=quant)
    sb = w.streams(stream + 1, n_frames)
    frames = [sb.frame(i, stream) for i in range(n_frames)]
    orc.lib()
    t0 = time.perf_counter()
    for f in frames:
        oc.infer_frame(f)
    dt = time.perf_counter() - t0
    n_full = (n_frames + w.expire_n - 1) // w.expire_n
    return n_frames / dt, dt, f"stream {stream}, frames 0-{n_frames - 1} ({n_full} full + {n_frames - n_full} cached)"


def reference_arm(args, w):
    """The oracle timed on the host cores, per the same metric.  Each step is a bounded
    sample: one frame of one stream."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import deepcache_oracle as orc
    ws, bs = w.weights()
    quant = orc.QUANT_BF16 if w.dtype == 1 else orc.QUANT_NONE
    oc = orc.OracleCache(w.width, w.height, w.layers, ws, bs, block=w.block, search_range=w.range,
                         search_kind=w.search, psnr_db=w.psnr_db, expire_n=w.expire_n, quant=quant)
    total = args.warmup + args.steps
    sb = w.streams(1, total)
    frames = [sb.frame(i, 0) for i in range(total)]
    for f in frames[:args.warmup]:
        oc.infer_frame(f)
    t0 = time.perf_counter()
    for f in frames[args.warmup:]:
        oc.infer_frame(f)
    dt = time.perf_counter() - t0
    fps = args.steps / dt
    cores = os.cpu_count()
    sample = f"one stream of the workload, one frame per step ({args.steps} timed frames after {args.warmup})"
    line = {"impl": "reference", "metric": METRIC, "value": fps, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": workload_config(w, 1, args.gpus),
            "cpu_baseline": {"value": fps, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": fps, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ---------------------------------------------------------------------------
# clocks
# ---------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "50"], stdout=subprocess.PIPE, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.perf_counter(), [v.strip() for v in line.split(",")]))

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        rows = [r for t, r in self.rows if t0 <= t <= t1] or [r for _, r in self.rows[-3:]]
        sm, smax, reasons = [], None, set()
        for r in rows:
            try:
                sm.append(float(r[0])); smax = float(r[1])
            except Exception:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": smax, "reasons": sorted(reasons),
                "samples": len(sm)}


# ---------------------------------------------------------------------------
# our arm
# ---------------------------------------------------------------------------
def gpu_arm(args, w):
    import torch
    import torch.distributed as dist
    from paper_1712_01670_b200 import binding as B
    from paper_1712_01670_b200 import sharding
    from paper_1712_01670_b200.engine import DeepCache

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.gpus > 1 and world != args.gpus:
        raise SystemExit("--gpus N > 1 needs torchrun with N ranks")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    # The cache works on the stream that is current when it is created.  A stream of raised priority lets the
    # inference kernels take the SMs ahead of the looked-ahead matcher, which runs on a lowest-priority stream.
    with torch.cuda.stream(torch.cuda.Stream(dev, priority=-1)):
        gpu_arm_on_stream(args, w, B, sharding, DeepCache, dist, rank, world, local, dev)


def reuse_copy_bench(args, B, DeepCache, rank, dev):
    """Reuse copy alone: one 3 -> 64 channel 3x3 layer at 224 x 224, bf16, S streams; six rectangles per stream cover
    about 79 % of the map, each displaced by its own vector.  dc_conv_partial runs the three steps of "Reuse"; the
    event profile separates the copy + bitmap kernel from the convolution of the rest."""
    import torch
    from paper_1712_01670_b200.synth import nets
    S = args.streams or 32
    H = W = 224
    nb = nets.NetBuilder(H, W)
    nb.conv(-1, 64, 3, 1, 1, 1)
    ws, bs = nets.random_weights(nb.layers, 5)
    dc = DeepCache(W, H, nb.layers, ws, bs, n_streams=S, block=16, search_range=8, dtype=B.DC_BF16, max_regions=8)
    g = np.random.Generator(np.random.PCG64(1712))
    regs = np.zeros((S, dc.max_regions, 6), np.int32)
    reused_px = 0
    cw, ch = W // 3, H // 2
    for s in range(S):
        for i in range(6):
            w_, h_ = cw - 8, ch - 12
            x0, y0 = (i % 3) * cw + int(g.integers(0, 9)), (i // 3) * ch + int(g.integers(0, 13))
            sx = min(max(x0 + int(g.integers(-8, 9)), 0), W - w_)
            sy = min(max(y0 + int(g.integers(-8, 9)), 0), H - h_)
            regs[s, i] = (x0, y0, w_, h_, sx, sy)
            reused_px += w_ * h_
    regs_d = torch.from_numpy(regs).to(dev)
    n_d = torch.full((S,), 6, dtype=torch.int32, device=dev)
    x = torch.rand((S, H, W, 3), device=dev).to(torch.bfloat16)
    maps = [torch.randn((S, H, W, 64), device=dev).to(torch.bfloat16) for _ in range(2)]
    for i in range(args.warmup):
        B.dc_conv_partial(dc.handle, 0, x, maps[i & 1], regs_d, n_d, maps[(i & 1) ^ 1])
    torch.cuda.synchronize()
    B.dc_cache_set_profiling(dc.handle, True)
    B.dc_cache_profile(dc.handle)
    for i in range(args.steps):
        B.dc_conv_partial(dc.handle, 0, x, maps[i & 1], regs_d, n_d, maps[(i & 1) ^ 1])
    torch.cuda.synchronize()
    prof = B.dc_cache_profile(dc.handle)
    status = dc.status()
    dc.close()
    ms = prof["classify_copy"][0] / max(1, prof["classify_copy"][1])
    bytes_per_launch = 2.0 * reused_px * 64 * 2
    peaks = measured_peaks()
    gbs = bytes_per_launch / (ms * 1e-3) / 1e9
    if rank == 0:
        print(json.dumps({"stage": "reuse copy + bitmaps (k_classify_copy), one 64-channel 224x224 bf16 layer",
                          "streams": S, "reuse_ratio": reused_px / (S * H * W), "ms_per_launch": ms,
                          "launches": prof["classify_copy"][1], "bytes_per_launch": bytes_per_launch,
                          "roofline_copy": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                            "frac": gbs / peaks["hbm_gbs"], "peak_source": f"hbm_gbs, {peaks['source']}"},
                          "conv_ms_per_launch": prof["conv"][0] / max(1, prof["conv"][1]), "status": status}))


def conv_layer_bench(args, B, DeepCache, rank, dev):
    """One convolution layer alone, every tile computed: CIN -> COUT channels on HW x HW maps, bf16, S streams."""
    import torch
    from paper_1712_01670_b200.synth import nets
    parts = [int(v) for v in args.conv_layer.split(",")]
    cin, cout, hw = parts[:3]
    k = parts[3] if len(parts) > 3 else 3
    S = args.streams or 32
    nb = nets.NetBuilder(hw, hw)
    first = nb.conv(-1, cin, 1, 1, 0)                    # stands in for the producer of the layer's input
    nb.conv(first, cout, k, 1, k // 2, 1)
    ws, bs = nets.random_weights(nb.layers, 9)
    dc = DeepCache(hw, hw, nb.layers, ws, bs, n_streams=S, block=16, search_range=4, dtype=B.DC_BF16)
    x = torch.randn((S, hw, hw, cin), device=dev).to(torch.bfloat16)
    out = torch.empty((S, hw, hw, cout), device=dev, dtype=torch.bfloat16)
    for _ in range(args.warmup):
        B.dc_conv_partial(dc.handle, 1, x, None, None, None, out)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        B.dc_conv_partial(dc.handle, 1, x, None, None, None, out)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    status = dc.status()
    dc.close()
    flops = 2.0 * S * hw * hw * cout * cin * k * k
    peaks = measured_peaks()
    tf = flops / (ms * 1e-3) / 1e12
    if rank == 0:
        print(json.dumps({"stage": f"convolution {cin} -> {cout}, {k}x{k}, {hw}x{hw} maps, bf16, all tiles", "streams": S,
                          "scheme": os.environ.get("DC_CONV_SCHEME", "tuned"), "ms_per_launch": ms, "tflops": tf,
                          "frac_burst": tf / peaks["bf16_tflops"], "frac_sustained": tf / peaks["bf16_tflops_sustained"],
                          "status": status}))


def gpu_arm_on_stream(args, w, B, sharding, DeepCache, dist, rank, world, local, dev):
    import torch
    if args.reuse_copy or args.conv_layer:
        (reuse_copy_bench if args.reuse_copy else conv_layer_bench)(args, B, DeepCache, rank, dev)
        if world > 1:
            dist.destroy_process_group()
        return
    S = args.streams or w.n_streams
    total = args.warmup + args.steps
    # every rank renders its own streams: global stream index = rank * S + s
    my = sharding.shard_streams(rank, world, S)
    sb_mine = w.streams(S, total, first=my[0]) if world > 1 else w.streams(S, total)
    frame_bytes = w.height * w.width * 3
    host = torch.empty((total, S, w.height, w.width, 3), dtype=torch.uint8).pin_memory()
    host_np = host.numpy()

    def render(job):
        s, i = job
        host_np[i, s] = sb_mine.streams[s].frame(i)
    with ThreadPoolExecutor(max_workers=min(16, os.cpu_count() or 4)) as ex:
        list(ex.map(render, [(s, i) for s in range(S) for i in range(total)]))
    dev_frames = host.to(dev, non_blocking=True)
    torch.cuda.synchronize()

    dc = DeepCache.from_workload(w, n_streams=S, device=f"cuda:{local}", skip_k=args.skip_k,
                                 cache_pool=args.cache_pool, region_mode=1 if args.per_block_regions else 0)
    pitch = w.width * 3
    last = w.layers[-1]
    out_bytes = S * last["out_h"] * last["out_w"] * last["cout"] * (2 if w.dtype == 1 else 4)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    if args.matcher_only:
        for i in range(1, args.warmup + 1):
            B.dc_cache_set_key(dc.handle, dev_frames[max(i - 1, 0)], pitch)
            B.dc_match_blocks(dc.handle, dev_frames[i], pitch)
        barrier()
        m0, m1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        m0.record()
        for i in range(args.warmup, total):
            B.dc_cache_set_key(dc.handle, dev_frames[max(i - 1, 0)], pitch)
            B.dc_match_blocks(dc.handle, dev_frames[i], pitch)
        m1.record()
        barrier()
        ms = m0.elapsed_time(m1) / args.steps
        if rank == 0:
            print(json.dumps({"stage": "matcher (key copy, frame copy, Steps 2-5)", "ms_per_step": ms, "streams": S,
                              "steps": args.steps, "warmup": args.warmup, "config": workload_config(w, S, world),
                              "algorithmic_gbs": 4.0 * frame_bytes * S / (ms * 1e-3) / 1e9}))
        dc.close()
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- device-resident timing: value ----
    # The loop a user runs: infer frame t, then announce frame t+1 so that its matching runs on a side stream
    # beside the convolutions of frame t (dc_lookahead_frame; results are identical without it).
    overlap = not args.no_lookahead

    def step(i):
        B.dc_infer_frame(dc.handle, dev_frames[i], pitch)
        if overlap and i + 1 < total:
            B.dc_lookahead_frame(dc.handle, dev_frames[i + 1], pitch)

    for i in range(args.warmup):
        step(i)
    barrier()
    launches0 = dc.launches()
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.25)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t0 = time.perf_counter()
    e0.record()
    for i in range(args.warmup, total):
        step(i)
    e1.record()
    barrier()
    t1 = time.perf_counter()
    ms = e0.elapsed_time(e1)
    clocks = sampler.stop(t0, t1)
    launches = dc.launches() - launches0
    status = dc.status()
    if status != B.DC_OK:
        raise SystemExit(f"device status {status}: {B.strerror(status)}")
    ms = sharding.max_over_ranks(ms, dev)
    value = sharding.aggregate_rate(S * args.steps, world, ms * 1e-3)

    # ---- the same K steps once more, one stream only and every launch bracketed by events: per-kernel
    #      durations for the rooflines are taken here, where kernels do not share the SMs ----
    dc.reset()
    for i in range(args.warmup):
        B.dc_infer_frame(dc.handle, dev_frames[i], pitch)
    barrier()
    B.dc_cache_set_profiling(dc.handle, True)
    B.dc_cache_profile(dc.handle)
    px0, cached0, full0 = B.dc_cache_counters(dc.handle, len(w.layers))
    s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s0.record()
    for i in range(args.warmup, total):
        B.dc_infer_frame(dc.handle, dev_frames[i], pitch)
    s1.record()
    barrier()
    serial_ms = sharding.max_over_ranks(s0.elapsed_time(s1), dev)
    prof = B.dc_cache_profile(dc.handle)
    B.dc_cache_set_profiling(dc.handle, False)
    px1, cached1, full1 = B.dc_cache_counters(dc.handle, len(w.layers))

    # ---- end to end through the host-buffer entry point ----
    e2e = None
    if not args.no_e2e:
        dc.reset()
        out_host = torch.empty(out_bytes, dtype=torch.uint8).pin_memory()
        for i in range(args.warmup):
            B.dc_infer_frame_host(dc.handle, host[i].data_ptr(), pitch, out_host.data_ptr())
        barrier()
        t0e = time.perf_counter()
        for i in range(args.warmup, total):
            if i + 1 < total:                  # the next step's input copy overlaps this step's compute
                B.dc_prefetch_frame_host(dc.handle, host[i + 1].data_ptr(), pitch)
            B.dc_infer_frame_host(dc.handle, host[i].data_ptr(), pitch, out_host.data_ptr())
        torch.cuda.synchronize()
        dte = time.perf_counter() - t0e
        dte = sharding.max_over_ranks(dte, dev)
        e2e = {"value": sharding.aggregate_rate(S * args.steps, world, dte), "unit": UNIT, "h2d_bytes_per_step": S * frame_bytes,
               "d2h_bytes_per_step": out_bytes}

    # ---- the same frames with the cache switched off (every frame computed in full): the paper's "no-cache" arm ----
    dc.close()
    nc = DeepCache.from_workload(w, n_streams=S, device=f"cuda:{local}", expire_n=1)
    for i in range(args.warmup):
        B.dc_infer_frame(nc.handle, dev_frames[i], pitch)
    barrier()
    n0, n1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n0.record()
    for i in range(args.warmup, total):
        B.dc_infer_frame(nc.handle, dev_frames[i], pitch)
    n1.record()
    barrier()
    no_cache_ms = sharding.max_over_ranks(n0.elapsed_time(n1), dev)
    no_cache = {"value": sharding.aggregate_rate(S * args.steps, world, no_cache_ms * 1e-3), "unit": UNIT,
                "ms_per_step": no_cache_ms / args.steps,
                "note": "same kernels, expire_n = 1: no matching, no reuse, every tile computed"}
    cache_bytes = nc.bytes()
    nc.close()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- rooflines from the event profile of the timed region ----
    peaks = measured_peaks()
    fpp = conv_flops_per_pixel(w.layers)
    n_cached, n_full = cached1 - cached0, full1 - full0
    useful_flops = 0.0
    reuse = {}
    for li, l in enumerate(w.layers):
        if l["kind"] != 0:
            continue
        all_px = l["out_h"] * l["out_w"] * S * (n_cached + n_full)
        reused = px1[li] - px0[li]
        useful_flops += fpp[li] * (all_px - reused)
        reuse[str(li)] = round(reused / max(1, l["out_h"] * l["out_w"] * S * max(1, n_cached)), 4)
    conv_ms, conv_n = prof["conv"]
    stage_ms = {k: round(v[0], 4) for k, v in prof.items()}
    stage_share = {k: round(v[0] / max(1e-9, sum(x[0] for x in prof.values())), 4) for k, v in prof.items()}
    bf16 = w.dtype == 1
    conv_tflops = useful_flops / (conv_ms * 1e-3) / 1e12 if conv_ms > 0 else 0.0
    # Which measured peak applies: the burst figure for a region that ran at full clock without a power cap, the
    # sustained one when the sampled clocks show the cap (long dense steps).  Both fractions are printed.
    capped = "sw_power_cap" in (clocks.get("reasons") or []) or \
             (clocks.get("sm_mhz") and clocks.get("sm_max_mhz") and clocks["sm_mhz"] < 0.9 * clocks["sm_max_mhz"])
    conv_peak = (peaks["bf16_tflops_sustained"] if capped else peaks["bf16_tflops"]) if bf16 else None
    conv_traffic, conv_traffic_from = captured_traffic("conv", w.index == 5 and S == 32 and bf16 and not args.cache_pool)
    roofline = {"kernel": "partial convolution (all conv launches of the timed region)",
                "bound": "tensor" if bf16 else "alu", "achieved": conv_tflops,
                "peak": conv_peak, "unit": "TFLOP/s", "frac": (conv_tflops / conv_peak) if conv_peak else None,
                "peak_source": f"{'bf16_tflops_sustained' if capped else 'bf16_tflops (burst)'}, {peaks['source']}; "
                               f"chosen by the clocks sampled in the timed region ({clocks.get('sm_mhz')} MHz, reasons {clocks.get('reasons')})",
                "frac_burst": (conv_tflops / peaks["bf16_tflops"]) if bf16 else None,
                "frac_sustained": (conv_tflops / peaks["bf16_tflops_sustained"]) if bf16 else None,
                "traffic": conv_traffic, "traffic_from": conv_traffic_from,
                "traffic_unit": "bytes per launch (dram read + write, ncu)",
                "launches": conv_n, "avg_launch_ms": conv_ms / max(1, conv_n),
                "flops_per_launch": useful_flops / max(1, conv_n)}
    # Reuse copy (Section 5 "Reuse", step 1): 2 x reused pixels x channels x element size over the time of the kernel
    # that also builds the bitmaps and dirty lists.  Meaningful where reuse is high (see bench.py --reuse-copy).
    elt = 2 if bf16 else 4
    copy_bytes = sum(2.0 * (px1[li] - px0[li]) * l["cout"] * elt for li, l in enumerate(w.layers)
                     if l["kind"] == 0 or (args.cache_pool and l["kind"] in (1, 6)))
    copy_ms, copy_n = prof["classify_copy"]
    copy_gbs = copy_bytes / (copy_ms * 1e-3) / 1e9 if copy_ms > 0 else 0.0
    roofline_copy = {"kernel": "reuse copy + bitmaps + dirty lists (k_classify_copy_all)", "bound": "hbm", "achieved": copy_gbs,
                     "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": copy_gbs / peaks["hbm_gbs"],
                     "peak_source": f"hbm_gbs, {peaks['source']}", "traffic": None, "launches": copy_n,
                     "bytes_per_launch": copy_bytes / max(1, copy_n),
                     "note": "little is reusable on this workload, so the kernel mostly classifies tiles; "
                             "bench.py --reuse-copy times the copy at 79 % reuse"}
    match_ms = prof["search"][0] + prof["verify"][0]
    match_bytes = 4.0 * frame_bytes * S * n_cached            # Step 2: cur + prev once; Step 4: both again
    match_gbs = match_bytes / (match_ms * 1e-3) / 1e9 if match_ms > 0 else 0.0
    match_traffic, match_traffic_from = captured_traffic("matcher", w.index == 5 and S == 32 and w.search == 1 and args.skip_k == 1)
    roofline_matcher = {"kernel": "block search + verify", "bound": "hbm", "achieved": match_gbs,
                        "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": match_gbs / peaks["hbm_gbs"],
                        "peak_source": f"hbm_gbs, {peaks['source']}",
                        "traffic": match_traffic, "traffic_from": match_traffic_from,
                        "traffic_unit": "bytes per batch-frame (search + verify kernels; dram read + write, ncu)",
                        "launches": prof["search"][1] + prof["verify"][1],
                        "bytes_per_frame_batch": 4.0 * frame_bytes * S,
                        "note": "Step 4 is credited with both frames for every block although blocks whose own best vector is M "
                                "are settled without reading pixels; step2_only credits and times Step 2 alone",
                        "step2_only": {"bytes_per_frame_batch": 2.0 * frame_bytes * S,
                                       "achieved": (2.0 * frame_bytes * S * n_cached / (prof["search"][0] * 1e-3) / 1e9) if prof["search"][0] > 0 else 0.0,
                                       "frac": (2.0 * frame_bytes * S * n_cached / (prof["search"][0] * 1e-3) / 1e9 / peaks["hbm_gbs"]) if prof["search"][0] > 0 else 0.0}}

    if w.search == 0:
        # Exhaustive search is plain integer arithmetic: every byte of every valid candidate takes one
        # absolute difference and one multiply-accumulate.  Both run as 4-byte SIMD operations at 16 lanes
        # per clock and SM sub-partition, on two pipes that work side by side, so the ceiling is
        # SMs x 4 x 16 x 4 bytes per clock.
        bw = np.minimum(w.block, w.width - np.arange(0, w.width, w.block))
        bh = np.minimum(w.block, w.height - np.arange(0, w.height, w.block))
        x0, y0 = np.arange(0, w.width, w.block), np.arange(0, w.height, w.block)
        nx = np.minimum(w.range, w.width - bw - x0) + np.minimum(w.range, x0) + 1      # valid dx per block column
        ny = np.minimum(w.range, w.height - bh - y0) + np.minimum(w.range, y0) + 1
        byte_ops = 3.0 * float((nx * bw).sum()) * float((ny * bh).sum()) * S * n_cached
        search_ms = prof["search"][0]
        alu_peak = 148 * 4 * 16 * 4 * 1.965e9 / 1e12
        ach = byte_ops / (search_ms * 1e-3) / 1e12 if search_ms > 0 else 0.0
        roofline_matcher = {"kernel": "exhaustive block search", "bound": "alu", "achieved": ach, "peak": alu_peak,
                            "unit": "T squared byte differences/s", "frac": ach / alu_peak,
                            "peak_source": "148 SMs x 4 sub-partitions x 16 lanes x 4 bytes x 1965 MHz", "traffic": None,
                            "launches": prof["search"][1], "ops_per_frame_batch": byte_ops / max(1, n_cached)}
    cpu_baseline = None
    if not args.no_cpu_baseline:
        fps, secs, what = run_oracle_sample(w, 20)             # about 12 s of host time on workload 5
        cpu_baseline = {"value": fps, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle",
                        "sample": what + f", {secs:.1f} s"}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if bf16 else "f32", "data": "synthetic",
            "config": dict(workload_config(w, S, world), skip_k=args.skip_k, cache_pool=bool(args.cache_pool),
                           regions="per_block" if args.per_block_regions else "global"), "clocks": clocks, "e2e": e2e, "gpu_launches": launches,
            "roofline": roofline, "roofline_matcher": roofline_matcher, "roofline_copy": roofline_copy, "cpu_baseline": cpu_baseline,
            "stage_ms": stage_ms, "stage_share": stage_share, "frames_cached": n_cached, "frames_full": n_full,
            "reuse_ratio_cached_frames": reuse, "cache_bytes": cache_bytes, "no_cache": no_cache,
            "serial": {"value": sharding.aggregate_rate(S * args.steps, world, serial_ms * 1e-3), "unit": UNIT,
                       "ms_per_step": serial_ms / args.steps,
                       "note": "same steps without dc_lookahead_frame and with per-launch events: source of stage_ms and the rooflines"},
            "lookahead": {"enabled": overlap, "main_stream_priority": -1, "side_stream_priority": 0}}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    from paper_1712_01670_b200.synth import configs
    w = configs.WORKLOADS[args.workload]()
    if args.grouped:
        if args.workload != 3:
            raise SystemExit("--grouped applies to workload 3 (the AlexNet trunk)")
        w = configs.alexnet_stream(grouped=True)
    if args.search:
        w.search = {"exhaustive": configs.SEARCH_ES, "diamond": configs.SEARCH_DS, "three_step": configs.SEARCH_TSS}[args.search]
    if args.impl == "reference":
        reference_arm(args, w)
    else:
        gpu_arm(args, w)


if __name__ == "__main__":
    main()
