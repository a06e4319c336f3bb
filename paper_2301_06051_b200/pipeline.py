"""Sequencing of the C-ABI calls for a whole backbone pass (no arithmetic here).

A DSVT backbone is a stack of blocks; all blocks of a stage share the two rotated set tables of their
frame, so a pass is: dsvt_partition_rotated (X and Y axis tables), then one dsvt_block per block,
and optionally dsvt_pool followed by a second stage on the pooled grid.  With hybrid windows a stage holds one
pair of tables per distinct (window, shift) and calls dsvt_partition_shifted for the displaced cuts.
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence

import torch

from . import api


class Stage:
    """Blocks on one grid.  By default all blocks share one window shape and the two rotated set tables of the
    frame; `block_windows` gives each block its own (window, shift) instead (hybrid window partition: another
    window size and a displaced cut between consecutive blocks), with one pair of tables per distinct entry."""

    def __init__(self, ctx: api.Context, blocks: Sequence[Sequence[Dict]], batch: int, grid, window, set_size: int,
                 precision: int, max_voxels: int, block_windows: Optional[Sequence] = None):
        self.ctx, self.batch, self.grid, self.window, self.set_size = ctx, batch, tuple(grid), tuple(window), set_size
        dev = ctx.device
        self.blocks = [[api.device_weights(l, precision, dev) for l in blk] for blk in blocks]
        cap = max(int(max_voxels), 1)

        def new_tables():
            return [api.SetTable(torch.empty((cap, set_size), dtype=torch.int32, device=dev),
                                 torch.zeros(1, dtype=torch.int32, device=dev),
                                 torch.empty(4 * cap + 4, dtype=torch.int32, device=dev), cap, set_size)
                    for _ in range(2)]

        specs = [(self.window, None)] * len(self.blocks) if block_windows is None else [
            (tuple(w), None if sh is None else tuple(sh)) for w, sh in block_windows]
        assert len(specs) == len(self.blocks)
        self.specs = specs
        self._new_tables = new_tables
        self.tables_of = self.new_table_set()
        self.tables = self.tables_of[specs[0]] if specs else new_tables()  # the first block's pair

    def new_table_set(self) -> Dict:
        """One pair of set tables per distinct (window, shift) of the stage's blocks."""
        out = {}
        for sp in self.specs:
            if sp not in out:
                out[sp] = self._new_tables()
        return out

    def partition(self, coords: torch.Tensor, ctx: Optional[api.Context] = None, tables_of: Optional[Dict] = None,
                  n_dev: Optional[torch.Tensor] = None):
        """Fills the stage's tables, or those of another table set, through the stage's context or another one.
        `n_dev`: the voxel count as a device int32 (coords then has the stage's capacity)."""
        ctx = self.ctx if ctx is None else ctx
        for (window, shift), tables in (self.tables_of if tables_of is None else tables_of).items():
            ctx.partition_rotated(coords, self.batch, self.grid, window, self.set_size, out=tuple(tables), shift=shift,
                                  n_dev=n_dev)

    def run_blocks(self, coords: torch.Tensor, x: torch.Tensor, y: torch.Tensor,
                   tables_of: Optional[Dict] = None, ctx: Optional[api.Context] = None) -> torch.Tensor:
        """Every block on tables that are already filled; the result ends up in y."""
        tables_of = self.tables_of if tables_of is None else tables_of
        ctx = self.ctx if ctx is None else ctx
        # one dsvt_layers call for the whole stage: X-axis table, Y-axis table of every block's window cut
        tabs, ws = [], []
        for blk, sp in zip(self.blocks, self.specs):
            t = tables_of[sp]
            tabs += [t[0], t[1]]
            ws += [blk[0], blk[1]]
        src = x
        for i in range(0, len(ws), api.MAX_CHAIN_LAYERS):
            ctx.layers(src, tabs[i:i + api.MAX_CHAIN_LAYERS], ws[i:i + api.MAX_CHAIN_LAYERS], y, coords=coords)
            src = y  # (coords: read by layers with a position bias)
        return y

    def forward(self, coords: torch.Tensor, x: torch.Tensor, y: torch.Tensor) -> torch.Tensor:
        """Partition (both axes of every distinct window cut) then every block; the result ends up in y."""
        self.partition(coords)
        return self.run_blocks(coords, x, y)


class FrameStream:
    """Runs frames that live in pinned host memory through a Stage with the copies off the critical path: frame
    k + 1 is uploaded and frame k - 1 downloaded while frame k's kernels run (one upload stream, the context's
    stream for the kernels, one download stream; `depth` sets of device buffers).  Every frame is still copied in,
    computed and copied out in full; only the waiting is overlapped.  With `partition_ahead` the set tables of
    frame k + 1 (which need its coordinates only) are built on a stream of their own through a second context,
    into that frame's own table set, while frame k's blocks run: the partition's short kernels fill the SMs a
    layer launch leaves idle towards its end instead of standing between two frames' layer launches.  With
    several `lanes`, consecutive frames are dealt out to that many compute streams (each with its own context), so
    that a frame's layer launch starts on SMs as other frames' launches leave them: frames are independent, and a
    launch of one CTA per SM whose tiles do not divide evenly leaves SMs idle towards its end.  `layer_ctas` caps
    the CTAs of every lane's layer launches (0: one per SM); with the lanes together asking for somewhat more CTAs
    than the GPU has SMs, each CTA takes more tiles per start-up and one is always waiting for an SM to come free."""

    def __init__(self, stage: Stage, max_voxels: int, C: int, depth: int = 2, partition_ahead: bool = True,
                 lanes: int = 1, layer_ctas: int = 0):
        self.stage, self.depth, self.lanes = stage, int(depth), int(lanes)
        assert self.lanes == 1 or (partition_ahead and self.depth >= 2 * self.lanes), \
            "several lanes need partition_ahead and two buffer sets per lane"
        ctx = stage.ctx
        dev = ctx.device
        if self.lanes == 1:  # the stage's own context and stream
            self.compute, self.ctxs = [ctx.stream], [ctx]
        else:  # every lane on a stream and a context of its own; `layer_ctas` caps their layer launches' CTAs
            self.compute = [torch.cuda.Stream(dev) for _ in range(self.lanes)]
            self.ctxs = [ctx.sibling(st) for st in self.compute]
            for c in self.ctxs:
                c.set_layer_ctas(layer_ctas)
        self.up, self.down = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
        self.prep = self.prep_ctx = None
        if partition_ahead:
            self.prep = torch.cuda.Stream(dev)
            self.prep_ctx = ctx.sibling(self.prep)
            self.tables = [stage.new_table_set() for _ in range(self.depth)]
            self.partitioned = [torch.cuda.Event() for _ in range(self.depth)]
        self.cap, self.C = max(int(max_voxels), 1), int(C)
        self.coords = self.x = self.y = None  # device copies of host frames: allocated by the first submit()
        self.uploaded = [torch.cuda.Event() for _ in range(self.depth)]
        self.computed = [torch.cuda.Event() for _ in range(self.depth)]
        self.downloaded = [torch.cuda.Event() for _ in range(self.depth)]
        self.count = 0

    def _streams(self):
        return self.compute + [self.up, self.down] + ([self.prep] if self.prep is not None else [])

    def fence(self, event: torch.cuda.Event) -> None:
        """Nothing submitted from now on starts before `event` has happened."""
        for st in self._streams():
            st.wait_event(event)

    def join(self, stream: torch.cuda.Stream) -> None:
        """Makes `stream` wait for everything submitted so far."""
        for st in self._streams():
            if st != stream:
                e = torch.cuda.Event()
                e.record(st)
                stream.wait_event(e)

    def submit_resident(self, coords: torch.Tensor, x: torch.Tensor, y: torch.Tensor) -> None:
        """Enqueues one frame that already lives in device memory (no copies): partition on the look-ahead stream,
        blocks on the frame's lane, result in y.  The caller rotates over `depth` sets of (coords, x, y): a set may
        be handed in again once `depth` - 1 other frames have been submitted after it."""
        assert self.prep is not None and self.depth % self.lanes == 0
        s = self.count % self.depth
        lane = self.count % self.lanes
        compute, ctx = self.compute[lane], self.ctxs[lane]
        if self.count >= self.depth:
            self.prep.wait_event(self.computed[s])  # the blocks that last read this table set are done
        with torch.cuda.stream(self.prep):
            self.stage.partition(coords, ctx=self.prep_ctx, tables_of=self.tables[s])
            self.partitioned[s].record(self.prep)
        compute.wait_event(self.partitioned[s])
        with torch.cuda.stream(compute):  # (the frame that last wrote y ran on this lane: same stream, in order)
            self.stage.run_blocks(coords, x, y, tables_of=self.tables[s], ctx=ctx)
            self.computed[s].record(compute)
        self.count += 1

    def launch_count(self) -> int:
        return sum(c.launch_count() for c in self.ctxs + ([self.prep_ctx] if self.prep_ctx is not None else []))

    def submit(self, coords_h: torch.Tensor, feats_h: torch.Tensor, out_h: torch.Tensor) -> None:
        """Enqueues one frame: coords_h int32 [n, 4], feats_h float32 [n, C], out_h float32 [n, C], all pinned host
        tensors that must stay untouched until `wait()` returns (out_h is written by then).  Does not block unless the
        caller is `depth` frames ahead of the device."""
        assert coords_h.is_pinned() and feats_h.is_pinned() and out_h.is_pinned(), "pinned host memory only"
        n = int(feats_h.shape[0])
        if self.x is None:
            dev = self.stage.ctx.device
            self.coords = [torch.empty((self.cap, 4), dtype=torch.int32, device=dev) for _ in range(self.depth)]
            self.x = [torch.empty((self.cap, self.C), dtype=torch.float32, device=dev) for _ in range(self.depth)]
            self.y = [torch.empty((self.cap, self.C), dtype=torch.float32, device=dev) for _ in range(self.depth)]
        s = self.count % self.depth
        lane = self.count % self.lanes
        compute, ctx = self.compute[lane], self.ctxs[lane]
        reuse = self.count >= self.depth
        with torch.cuda.stream(self.up):
            if reuse:
                self.up.wait_event(self.computed[s])   # the frame that last used these inputs has been computed
            c, x = self.coords[s][:n], self.x[s][:n]
            c.copy_(coords_h, non_blocking=True)
            x.copy_(feats_h, non_blocking=True)
            self.uploaded[s].record(self.up)
        compute.wait_event(self.uploaded[s])
        if reuse:
            compute.wait_event(self.downloaded[s])  # y[s] of that frame has reached the host
        y = self.y[s][:n]
        if self.prep is not None:
            self.prep.wait_event(self.uploaded[s])
            if reuse:
                self.prep.wait_event(self.computed[s])  # the blocks that last read this table set are done
            with torch.cuda.stream(self.prep):
                self.stage.partition(c, ctx=self.prep_ctx, tables_of=self.tables[s])
                self.partitioned[s].record(self.prep)
            compute.wait_event(self.partitioned[s])
        with torch.cuda.stream(compute):
            if self.prep is not None:
                self.stage.run_blocks(c, x, y, tables_of=self.tables[s], ctx=ctx)
            else:
                self.stage.forward(c, x, y)
            self.computed[s].record(compute)
        with torch.cuda.stream(self.down):
            self.down.wait_event(self.computed[s])
            out_h.copy_(y, non_blocking=True)
            self.downloaded[s].record(self.down)
        self.count += 1

    def wait(self) -> None:
        """Blocks until every submitted frame's output is in its host tensor."""
        self.down.synchronize()
        for st in self.compute:
            st.synchronize()
        self.up.synchronize()
        if self.prep is not None:
            self.prep.synchronize()

    def status_sync(self) -> int:
        """Synchronises and returns (and clears) the device status bits of every context the stream uses."""
        bits = 0
        for ctx in self.ctxs + ([self.prep_ctx] if self.prep_ctx is not None else []):
            bits |= ctx.status_sync()
        return bits


class Backbone:
    """One or two stages with an optional attention-style pooling step between them."""

    def __init__(self, cfg: Dict, device: int = 0, max_voxels: Optional[int] = None):
        n = int(max_voxels or cfg["n"])
        self.cfg = cfg
        self.precision = api.BF16_FP32ACC if cfg["precision"] == "bf16" else api.FP32
        grid, window = cfg["grid"], cfg["window"]
        nwin = cfg["batch"] * (-(-grid[0] // window[0])) * (-(-grid[1] // window[1])) * (-(-grid[2] // window[2]))
        bw = cfg.get("block_windows")
        if bw:  # displaced or larger windows: the largest window count of any cut
            for w, sh in bw:
                sh = sh or (0, 0, 0)
                cnt = cfg["batch"]
                for a in range(3):
                    cnt *= -(-(grid[a] + sh[a]) // w[a])
                nwin = max(nwin, cnt)
        max_windows = nwin
        self.pool_shape = cfg.get("pool_shape")
        if self.pool_shape:
            pg = [-(-grid[a] // self.pool_shape[a]) for a in range(3)]
            max_windows = max(max_windows, cfg["batch"] * pg[0] * pg[1] * pg[2])
        self.ctx = api.Context(n, max_windows, cfg["C"], device)
        self.stage1 = Stage(self.ctx, cfg["blocks"], cfg["batch"], grid, window, cfg["set_size"], self.precision, n,
                            block_windows=bw)
        self.stage2 = None
        if self.pool_shape:
            self.pool_w = api.device_weights(cfg["pool"], self.precision, self.ctx.device)
            self.pooled_grid = tuple(pg)
            self.stage2 = Stage(self.ctx, cfg["blocks_after_pool"], cfg["batch"], self.pooled_grid, window,
                                cfg["set_size"], self.precision, n)

    def forward_async(self, coords: torch.Tensor, x: torch.Tensor, y: torch.Tensor):
        """Enqueues the whole pass without a host read-back: the pooled voxel count stays on the device, the second
        stage's calls are sized by the capacity and read the count there.  Returns (coords_out, feats_out, num_out)
        at full capacity (rows past *num_out are not written); for a single stage (coords, y, None)."""
        self.stage1.forward(coords, x, y)
        if not self.stage2:
            return coords, y, None
        oc, of, num, _, _ = self.ctx.pool(coords, y, self.cfg["batch"], self.cfg["grid"], self.pool_shape, self.pool_w)
        self.stage2.partition(oc, n_dev=num)
        self.stage2.run_blocks(oc, of, of)
        return oc, of, num

    def forward(self, coords: torch.Tensor, x: torch.Tensor, y: torch.Tensor):
        """Returns (coords_out, feats_out, num_out) cut to the pooled voxel count (one read-back, after everything
        has been enqueued); for a single stage these are (coords, y, None)."""
        oc, of, num = self.forward_async(coords, x, y)
        if num is None:
            return oc, of, None
        m = int(num.item())
        return oc[:m], of[:m], num


class StagedBackbone:
    """Any number of stages with attention-style pooling between them (the voxel variant's layout: windows that
    shrink along z while pooling reduces the z extent).  cfg["stages"][i] = {"window", "blocks"}; cfg["pools"][i] =
    {"shape", "weights"} maps stage i's grid to stage i + 1's."""

    def __init__(self, cfg: Dict, device: int = 0):
        self.cfg = cfg
        n = int(cfg["n"])
        self.precision = api.BF16_FP32ACC if cfg["precision"] == "bf16" else api.FP32
        grids = [tuple(cfg["grid"])]
        for pl in cfg["pools"]:
            grids.append(tuple(-(-grids[-1][a] // pl["shape"][a]) for a in range(3)))
        self.grids = grids
        max_windows = 1
        for g, st in zip(grids, cfg["stages"]):
            w = st["window"]
            max_windows = max(max_windows, cfg["batch"] * (-(-g[0] // w[0])) * (-(-g[1] // w[1])) * (-(-g[2] // w[2])))
        for g in grids[1:]:  # pooling works on one region per cell of the next grid
            max_windows = max(max_windows, cfg["batch"] * g[0] * g[1] * g[2])
        self.ctx = api.Context(n, max_windows, cfg["C"], device)
        self.stages = [Stage(self.ctx, st["blocks"], cfg["batch"], g, st["window"], cfg["set_size"], self.precision, n)
                       for g, st in zip(grids, cfg["stages"])]
        self.pool_w = [api.device_weights(pl["weights"], self.precision, self.ctx.device) for pl in cfg["pools"]]

    def forward(self, coords: torch.Tensor, x: torch.Tensor, on_step=None):
        """Returns (coords, feats) of the last stage.  on_step(tag), if given, is called after every call group."""
        feats, num = x, None  # num: the current stage's voxel count on the device (None: all of coords)
        for i, stage in enumerate(self.stages):
            y = torch.empty_like(feats)
            stage.partition(coords, n_dev=num)
            if on_step:
                on_step("s%d_partition" % i)
            stage.run_blocks(coords, feats, y)
            if on_step:
                on_step("s%d_blocks" % i)
            feats = y
            if i < len(self.pool_w):
                # (no read-back: the next stage is sized by the capacity and reads the pooled count on the device)
                coords, feats, num, _, _ = self.ctx.pool(coords, feats, self.cfg["batch"], self.grids[i],
                                                         self.cfg["pools"][i]["shape"], self.pool_w[i], n_dev=num)
                if on_step:
                    on_step("s%d_pool" % i)
        if num is not None:  # one read-back at the end, to cut the results to size
            m = int(num.item())
            coords, feats = coords[:m], feats[:m]
        return coords, feats
