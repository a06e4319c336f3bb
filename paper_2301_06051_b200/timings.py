"""Per-configuration device timings of the path: partition (both axes), blocks, pooling, whole backbone.

    python -m paper_2301_06051_b200.timings [--configs 1 2 3 4 5] [--steps 20] [--hybrid] [--rpb] [--bev]

One JSON line per configuration.  Times are CUDA-event medians over `steps` passes on synthetic frames that are
resident in HBM; a 256 MiB write flushes L2 before every pass.  bench.py measures the headline configuration under
its full contract; this tool is the per-configuration table.
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

import dsvt_inputs as di
from . import api, pipeline


def time_staged(cfg, steps: int, device: int = 0):
    """Configurations with a `stages` list (the voxel variant's layout)."""
    dev = torch.device("cuda", device)
    bb = pipeline.StagedBackbone(cfg, device=device)
    coords = torch.from_numpy(cfg["coords"]).to(dev)
    x = torch.from_numpy(cfg["feats"]).to(dev)
    flush = torch.empty(64 * 1024 * 1024, dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream(dev)
    rec = []
    for it in range(3 + steps):
        flush.zero_()
        marks = []

        def on_step(tag):
            e = torch.cuda.Event(enable_timing=True)
            e.record(stream)
            marks.append((tag, e))

        on_step("start")
        oc, of = bb.forward(coords, x, on_step)
        rec.append(marks)
    torch.cuda.synchronize(dev)
    if bb.ctx.status_sync() != 0:
        raise SystemExit("device status word is not clean")
    spans = {}
    for r in rec[3:]:
        for (t0, e0), (t1, e1) in zip(r[:-1], r[1:]):
            spans.setdefault(t1, []).append(e0.elapsed_time(e1))
        spans.setdefault("backbone", []).append(r[0][1].elapsed_time(r[-1][1]))
    out = {"config": cfg["id"], "name": cfg["name"], "voxels": cfg["n"], "precision": cfg["precision"],
           "voxels_out": int(oc.shape[0])}
    out.update({"t_%s_ms" % k: float(np.median(v)) for k, v in spans.items()})
    out["frames_per_s"] = cfg["batch"] / (out["t_backbone_ms"] * 1e-3)
    return out


def time_bev(cid: int, steps: int, device: int = 0):
    """dsvt_bev_scatter on the configuration's frame (its input features stand in for the backbone's output): the
    whole call (cell map clear + mark + dense writer), both layouts; bytes = the map written + features and coords read."""
    cfg = di.make_config(cid)
    dev = torch.device("cuda", device)
    ctx = api.Context(cfg["n"], 8, cfg["C"], device=device)
    coords = torch.from_numpy(cfg["coords"]).to(dev)
    x = torch.from_numpy(cfg["feats"]).to(dev)
    flush = torch.empty(64 * 1024 * 1024, dtype=torch.float32, device=dev)
    out = {"config": cid, "name": cfg["name"], "voxels": cfg["n"], "grid": list(cfg["grid"]), "C": cfg["C"]}
    for tag, last in (("channels_first", False), ("channels_last", True)):
        m = ctx.bev_scatter(coords, x, cfg["batch"], cfg["grid"], last)
        ts = []
        for it in range(3 + steps):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            ctx.bev_scatter(coords, x, cfg["batch"], cfg["grid"], last, out=m)
            e1.record()
            torch.cuda.synchronize(dev)
            ts.append(e0.elapsed_time(e1))
        t = float(np.median(ts[3:]))
        nbytes = 4 * (m.numel() + x.numel() + coords.numel())
        out.update({"t_%s_ms" % tag: t, "gbs_%s" % tag: nbytes / t * 1e-6})
        del m
    out["map_mb"] = 4e-6 * cfg["batch"] * cfg["C"] * int(np.prod(cfg["grid"]))
    if ctx.status_sync() != 0:
        raise SystemExit("device status word is not clean")
    return out


def add_position_bias(cfg, seed: int = 0):
    """Gives every layer of a single-stage configuration a random relative position bias table for its window."""
    rng = np.random.default_rng(seed)
    wins = [cfg["window"]] + [w for w, _ in cfg.get("block_windows") or []]
    L, W, H = (max(w[a] for w in wins) for a in range(3))  # one table extent that covers every block's windows
    for blk in cfg["blocks"]:
        for layer in blk:
            layer["rpb"] = rng.standard_normal((cfg["heads"], (2 * L - 1) * (2 * W - 1) * (2 * H - 1))).astype(np.float32)
            layer["rpb_extent"] = (L, W, H)


def time_config(cid: int, steps: int, device: int = 0, hybrid: bool = False, rpb: bool = False):
    cfg = di.make_config(cid)
    if cfg.get("stages"):
        return time_staged(cfg, steps, device)
    dev = torch.device("cuda", device)
    if hybrid:
        # hybrid window partition (Sec. 3.2): every second block works on windows twice as large in x and y,
        # cut with a displacement of one original window
        w = cfg["window"]
        big = (2 * w[0], 2 * w[1], w[2])
        cfg["block_windows"] = [(w, None) if i % 2 == 0 else (big, (w[0], w[1], 0)) for i in range(len(cfg["blocks"]))]
    if rpb:
        add_position_bias(cfg)
    bb = pipeline.Backbone(cfg, device=device)
    coords = torch.from_numpy(cfg["coords"]).to(dev)
    x = torch.from_numpy(cfg["feats"]).to(dev)
    y = torch.empty_like(x)
    flush = torch.empty(64 * 1024 * 1024, dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream(dev)
    rec = []

    def mark(tag):
        e = torch.cuda.Event(enable_timing=True)
        e.record(stream)
        rec[-1].append((tag, e))

    def run_stage(stage, c, src, dst, tag):
        stage.partition(c)
        mark(tag + "partition")
        for blk, sp in zip(stage.blocks, stage.specs):
            t = stage.tables_of[sp]  # (hybrid windows: every block runs on the tables of its own cut)
            bb.ctx.block(src, t[0], t[1], blk, dst, coords=c)
            src = dst
        mark(tag + "blocks")

    m = cfg["n"]
    for it in range(3 + steps):
        flush.zero_()
        rec.append([])
        mark("start")
        run_stage(bb.stage1, coords, x, y, "s1_")
        if bb.stage2:
            oc, of, num, _, _ = bb.ctx.pool(coords, y, cfg["batch"], cfg["grid"], bb.pool_shape, bb.pool_w)
            mark("pool")
            m = int(num.item())  # the pooled voxel count sizes the second stage's tensors
            mark("readback")
            run_stage(bb.stage2, oc[:m], of[:m], of[:m], "s2_")
    torch.cuda.synchronize(dev)
    if bb.ctx.status_sync() != 0:
        raise SystemExit("device status word is not clean")
    spans = {}
    for r in rec[3:]:
        for (t0, e0), (t1, e1) in zip(r[:-1], r[1:]):
            spans.setdefault(t1, []).append(e0.elapsed_time(e1))
        spans.setdefault("backbone", []).append(r[0][1].elapsed_time(r[-1][1]))
    med = {k: float(np.median(v)) for k, v in spans.items()}
    nb1 = len(bb.stage1.blocks)
    out = {"config": cid, "name": cfg["name"] + (" + hybrid windows" if hybrid else "") + (" + position bias" if rpb else ""), "voxels": cfg["n"], "precision": cfg["precision"],
           "sets": int(bb.stage1.tables[0].num_sets.item()),
           "t_partition_ms": med["s1_partition"], "t_block_ms": med["s1_blocks"] / nb1,
           "voxels_per_s_per_block": cfg["n"] / (med["s1_blocks"] / nb1 * 1e-3),
           "t_backbone_ms": med["backbone"], "frames_per_s": cfg["batch"] / (med["backbone"] * 1e-3)}
    if bb.stage2:
        nb2 = len(bb.stage2.blocks)
        out.update({"t_pool_ms": med["pool"], "pooled_voxels": m, "t_partition2_ms": med["s2_partition"],
                    "t_block2_ms": med["s2_blocks"] / nb2})
    return out


def main():
    ap = argparse.ArgumentParser(description=__doc__)
    ap.add_argument("--configs", type=int, nargs="+", default=list(di.CONFIG_IDS),
                    help="1..5; 6 = the nuScenes-shaped extra (windows 30 x 30, set size 90, C=128); 7 = DSVT-V stage layout")
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--hybrid", action="store_true",
                    help="alternate the configuration's windows with doubled, displaced ones (single-stage configurations)")
    ap.add_argument("--rpb", action="store_true",
                    help="give every layer a relative position bias table for its window (single-stage configurations)")
    ap.add_argument("--bev", action="store_true", help="time the BEV projection of each configuration's frame instead")
    args = ap.parse_args()
    api.load()
    for cid in args.configs:
        if args.bev:
            print(json.dumps(time_bev(cid, args.steps)), flush=True)
        else:
            print(json.dumps(time_config(cid, args.steps, hybrid=args.hybrid, rpb=args.rpb)), flush=True)


if __name__ == "__main__":
    main()
