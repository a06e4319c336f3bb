#!/usr/bin/env python
"""Benchmark of the DSVT hot path on synthetic LiDAR-shaped frames.

A step is one pass of the whole path over one frame: rotated set partition (both sort axes), then
every DSVT block of the backbone (configuration 2: 32,000 pillars on 468 x 468, C = 192, 8 heads,
set size 36, four blocks of two layers with MLP and LayerNorm, bfloat16 weights, fp32 accumulate).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config 2]

Prints one JSON line (rank 0).  With N > 1 (torchrun) every rank runs its own frame: the path shards
by frame with no collective, so scaling is weak.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "voxels/sec per DSVT block (partition amortised over the backbone); frames_per_sec = backbone frames/sec"
L2_FLUSH_BYTES = 256 << 20


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# dram__bytes_read.sum + dram__bytes_write.sum of one fused-layer launch at configuration 2, from the ncu capture
# summarised in profiles/layer_tc_kernel_config2.md (25.63 MB read + 0.06 MB written: the output stays in L2).
LAYER_DRAM_BYTES_PER_LAUNCH = 25.69e6


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.proc, self.idx, self.rows, self.thread = None, gpu_index, [], None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.perf_counter(), line))

    def start(self, wait_s: float = 5.0):
        """Starts nvidia-smi and returns once its first sample has arrived (or after wait_s)."""
        import threading

        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.idx), "--query-gpu=" + self.QUERY,
                                          "--format=csv,noheader,nounits", "-lms", "50"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True, bufsize=1)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()
        t0 = time.perf_counter()
        while not self.rows and time.perf_counter() - t0 < wait_s and self.proc.poll() is None:
            time.sleep(0.01)

    def stop(self, t_begin: float, t_end: float):
        """Summary of the samples taken in [t_begin, t_end] (perf_counter times of the timed region); if the
        region was shorter than one sampling period, of the samples closest to it."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"], "samples": 0}
        time.sleep(0.06)  # one more sampling period, so that a short region is bracketed
        self.proc.terminate()
        try:
            self.proc.wait(timeout=10)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        if self.thread is not None:
            self.thread.join(timeout=5)
        inside = [r for r in self.rows if t_begin <= r[0] <= t_end]
        note = "all samples inside the timed region"
        if not inside and self.rows:
            mid = 0.5 * (t_begin + t_end)
            inside = sorted(self.rows, key=lambda r: abs(r[0] - mid))[:2]
            note = "timed region shorter than the 50 ms sampling period: the two samples closest to it"
        sm, mx, reasons = [], [], set()
        for _, line in inside:
            f = [t.strip() for t in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm), "note": note}


def _dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def algorithmic_flops_per_layer(rowoff: np.ndarray, C: int, hidden: int) -> float:
    """Projections 8 C^2 + MLP 4 C hidden per voxel, attention 4 m^2 C per set of m distinct voxels."""
    m = np.diff(rowoff).astype(np.float64)
    n = float(rowoff[-1])
    return n * (8.0 * C * C + 4.0 * C * hidden) + 4.0 * C * float((m * m).sum())


def max_over_ranks(values, device=None):
    """Element-wise maximum of a list of floats over all ranks (identity when not distributed)."""
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def job_throughput(world: int, units_per_rank: float, ms_per_step: float) -> float:
    """Whole-job units per second: every rank processes units_per_rank per step (weak scaling), and a
    step takes as long as the slowest rank."""
    return world * units_per_rank / (ms_per_step * 1e-3)


def workload_name(cid: int, cfg) -> str:
    """The `config.workload` string: the same for both arms."""
    return "config %d (%s): %d voxels, grid %s, window %s, set size %d, C=%d, %d blocks x 2 layers" % (
        cid, cfg["name"], cfg["n"], cfg["grid"], cfg["window"], cfg["set_size"], cfg["C"], len(cfg["blocks"]))


def run_reference(args):
    """The CPU oracle as it stands, on a bounded sample of the same workload (rank 0 only)."""
    rank, _, world = _dist_env()
    if rank != 0:
        return
    import dsvt_inputs as di
    from oracle import ref

    cores = ref.max_threads()
    ref.set_threads(cores)
    cfg = di.make_config(args.config)
    n_s = min(cfg["n"], 1200)
    p = ref.partition(cfg["coords"], cfg["batch"], cfg["grid"], cfg["window"], cfg["set_size"], 0)
    # whole windows in window order until about n_s voxels
    w_end = int(np.searchsorted(p.win_start, n_s))
    sel = np.sort(p.perm[: p.win_start[w_end]])
    cs, fs = cfg["coords"][sel], cfg["feats"][sel].astype(np.float64)

    def step():
        t0 = ref.partition(cs, cfg["batch"], cfg["grid"], cfg["window"], cfg["set_size"], 0)
        t1 = ref.partition(cs, cfg["batch"], cfg["grid"], cfg["window"], cfg["set_size"], 1)
        x = fs
        for blk in cfg["blocks"]:
            x = ref.block(x, t0.set_table, t1.set_table, blk)
        return x

    for _ in range(args.warmup):
        step()
    t = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = (time.perf_counter() - t) / args.steps
    value = sel.shape[0] * len(cfg["blocks"]) / dt
    sample = "%d voxels (whole windows) of config %d through partition + %d blocks per step" % (
        sel.shape[0], args.config, len(cfg["blocks"]))
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "voxels/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(args.config, cfg), "sample": sample},
        "cpu_baseline": {"value": value, "unit": "voxels/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "voxels/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_ours(args):
    import torch

    import dsvt_inputs as di
    from paper_2301_06051_b200 import api, pipeline

    rank, local_rank, world = _dist_env()
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    api.load()  # no fallback: a missing library is an error

    cfg = di.make_config(args.config)
    if cfg.get("pool_shape"):
        raise SystemExit("bench.py times single-stage configurations (1-4)")
    n, C, nb = cfg["n"], cfg["C"], len(cfg["blocks"])
    bb = pipeline.Backbone(cfg, device=local_rank)
    ctx, stage = bb.ctx, bb.stage1
    coords_h = torch.from_numpy(cfg["coords"]).pin_memory()
    feats_h = torch.from_numpy(cfg["feats"]).pin_memory()
    out_h = torch.empty((n, C), dtype=torch.float32).pin_memory()
    coords = coords_h.to(dev)
    x = feats_h.to(dev)
    y = torch.empty_like(x)
    flush = torch.empty(L2_FLUSH_BYTES // 4, dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream(dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    def step_device():
        stage.forward(coords, x, y)

    # end to end: every step uploads its frame from pinned host memory, runs the step and downloads the result;
    # pipeline.FrameStream overlaps the copies and the partition of neighbouring steps with the kernels and deals
    # the steps out to four compute streams (eight sets of device buffers)
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    LANES, R = 4, 8                 # compute streams, rotating sets of buffers
    lane_ctas = (sms + 2) // 3      # CTAs per layer launch: the four lanes ask for more CTAs than there are SMs
    frames = pipeline.FrameStream(stage, n, C, depth=R, lanes=LANES, layer_ctas=lane_ctas)
    outs_h = [out_h] + [torch.empty((n, C), dtype=torch.float32).pin_memory() for _ in range(R - 1)]

    def run_e2e(steps):
        for k in range(steps):
            frames.submit(coords_h, feats_h, outs_h[k % R])
        frames.wait()

    for _ in range(max(args.warmup, 3)):
        flush.zero_()
        step_device()
    barrier()
    if ctx.status_sync() != 0:
        raise SystemExit("device status word is not clean after warm-up")

    # ---- timed region: K steps, inputs resident in HBM, through the pipeline a stream of frames runs in: the next
    # step's partition on its own stream, consecutive steps dealt out to four compute streams whose layer launches
    # take a third of the SMs each.  The steps rotate over eight sets of (coords, x, y), 397 MB at configuration 2:
    # larger than L2. ----
    cs = [coords] + [coords.clone() for _ in range(R - 1)]
    xs = [x] + [x.clone() for _ in range(R - 1)]
    ys = [torch.empty_like(x) for _ in range(R)]
    resident = pipeline.FrameStream(stage, n, C, depth=R, lanes=LANES, layer_ctas=lane_ctas)
    for k in range(2 * R):
        resident.submit_resident(cs[k % R], xs[k % R], ys[k % R])
    barrier()
    if resident.status_sync() != 0:
        raise SystemExit("device status word is not clean after the pipeline's warm-up")
    ev_begin, ev_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local_rank)
    sampler.start()
    launches0 = resident.launch_count()
    barrier()
    t_begin = time.perf_counter()
    ev_begin.record(stream)
    resident.fence(ev_begin)
    for k in range(args.steps):
        resident.submit_resident(cs[k % R], xs[k % R], ys[k % R])
    resident.join(stream)
    ev_end.record(stream)
    barrier()
    t_end = time.perf_counter()
    launches = resident.launch_count() - launches0
    clocks = sampler.stop(t_begin, t_end)
    total_ms = float(ev_begin.elapsed_time(ev_end))
    if resident.status_sync() != 0:
        raise SystemExit("device status word is not clean after the timed region")

    # ---- one step at a time on one stream, L2 flushed (outside the events) before each: the latency of a step and
    # its parts (partition; all blocks as one chained launch, which the roofline figure is taken from) ----
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    barrier()
    for k in range(args.steps):
        flush.zero_()
        e = ev[k]
        e[0].record(stream)
        stage.partition(coords)
        e[1].record(stream)
        stage.run_blocks(coords, x, y)
        e[2].record(stream)
    barrier()
    t_step = np.array([e[0].elapsed_time(e[2]) for e in ev])  # ms
    t_part = np.array([e[0].elapsed_time(e[1]) for e in ev])
    t_chain = np.array([e[1].elapsed_time(e[2]) for e in ev])
    # the same blocks as one launch per block (dsvt_block), for comparison
    evb = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(args.steps)]
    yb = torch.empty_like(y)
    for k in range(args.steps):
        flush.zero_()
        evb[k][0].record(stream)
        src = x
        for blk in stage.blocks:
            ctx.block(src, stage.tables[0], stage.tables[1], blk, yb)
            src = yb
        evb[k][1].record(stream)
    barrier()
    t_blockwise = np.array([e[0].elapsed_time(e[1]) for e in evb])
    if not torch.equal(yb, y):
        raise SystemExit("block-by-block outputs differ from the chained launch")
    if any(not torch.equal(o, y) for o in ys):
        raise SystemExit("pipelined outputs differ from the one-step-at-a-time run")

    # ---- end to end through the public API with pinned host buffers ----
    run_e2e(R)
    barrier()
    e_steps = max(3, min(args.steps, 200))  # (the first upload and the last download are not overlapped)
    t0 = time.perf_counter()
    run_e2e(e_steps)
    barrier()
    e2e_ms = (time.perf_counter() - t0) * 1e3 / e_steps
    if any(not torch.equal(o, outs_h[0]) for o in outs_h[1:]) or not torch.equal(outs_h[0], y.cpu()):
        raise SystemExit("end-to-end outputs differ from the device-resident run")
    if frames.status_sync() != 0:
        raise SystemExit("device status word is not clean after the end-to-end steps")

    total_ms, e2e_ms = max_over_ranks([total_ms, e2e_ms], device=dev)
    if ctx.status_sync() != 0:
        raise SystemExit("device status word is not clean after the timed region")
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    ms_per_step = total_ms / args.steps
    value = job_throughput(world, n * nb, ms_per_step)
    peaks = _peaks()
    # dominant kernel: the fused layer kernel, two launches per block
    S = int(stage.tables[0].num_sets.item())
    fl = [algorithmic_flops_per_layer(stage.tables[a].set_rowoff[: S + 1].cpu().numpy(), C, cfg["hidden"])
          for a in (0, 1)]
    flops_per_launch = nb * (fl[0] + fl[1])  # one launch runs every layer of the stage
    launch_ms = float(t_chain.mean())
    achieved = flops_per_launch / (launch_ms * 1e-3) / 1e12
    pad = 1.0 - n / (S * cfg["set_size"])

    # ---- CPU oracle on a bounded sample (reported baseline, not a target) ----
    from oracle import ref

    cores = ref.max_threads()
    ref.set_threads(cores)
    t0 = time.perf_counter()
    p0 = ref.partition(cfg["coords"], cfg["batch"], cfg["grid"], cfg["window"], cfg["set_size"], 0)
    p1 = ref.partition(cfg["coords"], cfg["batch"], cfg["grid"], cfg["window"], cfg["set_size"], 1)
    xr = cfg["feats"]
    for blk in cfg["blocks"]:
        xr = ref.block(xr, p0.set_table, p1.set_table, blk)
    cpu_s = time.perf_counter() - t0
    cpu = {"value": n * nb / cpu_s, "unit": "voxels/s", "cores": cores, "kind": "oracle",
           "sample": "the whole frame (%d voxels): both partitions + all %d blocks, one pass, %.1f s wall"
                     % (n, nb, cpu_s)}

    print(json.dumps({
        "metric": METRIC, "value": value, "unit": "voxels/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if cfg["precision"] == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": workload_name(args.config, cfg),
                   "l2": "timed steps rotate over %d sets of inputs and outputs (%d MB, larger than L2); the "
                         "one-step-at-a-time figures: L2 flushed by a %d MiB write before every step"
                         % (R, R * (2 * x.numel() + coords.numel()) * 4 // 1000000, L2_FLUSH_BYTES >> 20),
                   "pipeline": "inputs resident in HBM; the next step's partition on its own stream, consecutive "
                               "steps dealt out to %d compute streams, %d CTAs per layer launch; CUDA events around "
                               "all K steps" % (LANES, lane_ctas),
                   "num_sets": S, "pad_ratio": pad, "frames_per_rank": 1},
        "frames_per_sec": world / (ms_per_step * 1e-3),
        "step_latency_ms": float(t_step.mean()),
        "t_partition_ms": float(t_part.mean()), "t_block_ms": launch_ms / nb,
        "t_block_ms_one_launch_per_block": float(t_blockwise.mean()) / nb,
        "clocks": clocks,
        "e2e": {"value": job_throughput(world, n * nb, e2e_ms), "unit": "voxels/s", "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": int(coords_h.numel() * 4 + feats_h.numel() * 4),
                "d2h_bytes_per_step": int(out_h.numel() * 4), "steps": e_steps,
                "how": "pipeline.FrameStream: per step one upload, one backbone pass, one download; copies of "
                       "neighbouring steps overlap the kernels, the next step's partition runs on its own stream "
                       "under the current step's layer launches, consecutive steps dealt out to four compute "
                       "streams; wall clock over all steps"},
        "gpu_launches": int(launches),
        "roofline": {"kernel": "fused DSVT layer", "bound": "tensor", "achieved": achieved,
                     "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": achieved / peaks["bf16_tflops"],
                     "frac_of_sustained": achieved / peaks["bf16_tflops_sustained"], "peak_source": peaks["source"],
                     "flops_per_launch": flops_per_launch, "ms_per_launch": launch_ms,
                     "layers_per_launch": 2 * nb,
                     "timing": "launch duration from the one-step-at-a-time run (a launch alone on the GPU)",
                     "achieved_in_pipeline": flops_per_launch / (ms_per_step * 1e-3) / 1e12,
                     "traffic": LAYER_DRAM_BYTES_PER_LAUNCH if args.config == 2 else None},
        "cpu_baseline": cpu,
    }))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2)
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
