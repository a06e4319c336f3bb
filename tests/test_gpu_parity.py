"""CUDA path vs the CPU oracle, through the C ABI (ctypes binding).  All tests need a B200."""
import numpy as np
import pytest
import torch

import dsvt_inputs as di
from gpu_helpers import check_close, dev, precision_of, row_rel_error, rowoff_of, table_np, upload_table

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gpu():
    from paper_2301_06051_b200 import api

    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    api.load()  # raises if the CUDA library has not been built: there is no fallback
    return api


PLAN_PACKED = 0x40000000  # flag on the tile count of a plan over a reordering of the sets


def _nwin(batch, grid, window):
    return batch * int(np.prod([-(-g // w) for g, w in zip(grid, window)]))


# ------------------------------------------------------------------------------------------------
# partition: bit-exact
# ------------------------------------------------------------------------------------------------
def _compare_table(t, ref, n, axis, extras=True):
    tbl, ro = table_np(t)
    assert tbl.shape == ref.set_table.shape, (axis, tbl.shape, ref.set_table.shape)
    assert np.array_equal(tbl, ref.set_table), axis
    assert np.array_equal(ro, rowoff_of(ref.set_table)), axis
    # tile plan behind the row offsets: whole sets in tiles of at most 128 rows, over a reordering of the sets that
    # needs fewer tiles than the greedy packing in table order (or in table order, where no reordering was found)
    tiles = None
    cap = t.cap_sets
    full = t.set_rowoff.cpu().numpy()
    plan = full[cap + 1:]
    S = tbl.shape[0]
    sizes = np.diff(ro)
    greedy, s = 0, 0
    while s < S:
        e = s + 1
        while e < S and ro[e + 1] - ro[s] <= 128:
            e += 1
        s = e
        greedy += 1
    if S > 24576:
        assert plan[0] == -1
    elif S > 0:
        T = int(plan[0]) & ~PLAN_PACKED
        e = plan[1:2 + T]
        fewest = -(-int(ro[S]) // 128)  # (a reordered plan within an eighth of this is taken without looking further)
        assert T <= max(greedy, fewest + fewest // 8) and e[0] == 0 and e[T] == S and np.all(np.diff(e) > 0), axis
        if int(plan[0]) & PLAN_PACKED:
            order = full[2 * cap + 3: 2 * cap + 3 + S]
            prow = full[3 * cap + 3: 3 * cap + 4 + S]
            assert np.array_equal(np.sort(order), np.arange(S)), axis
            assert np.array_equal(prow, np.concatenate([[0], np.cumsum(sizes[order])])), axis
        else:
            prow = ro
        assert np.all(prow[e[1:]] - prow[e[:-1]] <= 128), axis
        tiles = (T, greedy)
    if extras:
        assert np.array_equal(t.perm[:n].cpu().numpy(), ref.perm)
        assert np.array_equal(t.win_count.cpu().numpy(), ref.win_count)
        assert np.array_equal(t.win_start.cpu().numpy(), ref.win_start)
        assert np.array_equal(t.win_setoff.cpu().numpy(), ref.win_setoff)
    return tiles


def _check_partition(gpu, oracle, coords, batch, grid, window, tau, ctx=None):
    """dsvt_partition per axis and dsvt_partition_rotated, both against the oracle."""
    n = coords.shape[0]
    ctx = ctx or gpu.Context(max(n, 1), _nwin(batch, grid, window), 64)
    dc = dev(coords)
    refs = [oracle.partition(coords, batch, grid, window, tau, axis) for axis in (0, 1)]
    for axis in (0, 1):
        t = ctx.partition(dc, batch, grid, window, tau, axis, extras=True)
        assert ctx.status_sync() == 0
        _compare_table(t, refs[axis], n, axis)
    both = ctx.partition_rotated(dc, batch, grid, window, tau)
    assert ctx.status_sync() == 0
    for axis in (0, 1):
        tiles = _compare_table(both[axis], refs[axis], n, axis, extras=False)
    return ctx, tiles


@pytest.mark.parametrize("cid", [1, 2, 3, 4, 5, 6])
def test_partition_bit_exact_on_every_config(gpu, oracle, cid):
    cfg = di.make_config(cid, with_feats=False)
    _, tiles = _check_partition(gpu, oracle, cfg["coords"], cfg["batch"], cfg["grid"], cfg["window"], cfg["set_size"])
    if cid >= 2:  # LiDAR-shaped frames: the reordered plan saves tiles over the packing in table order
        print("config %d: %d tiles (%d in table order)" % (cid, tiles[0], tiles[1]))
        assert tiles[0] < tiles[1] and (cid == 5 or tiles[0] <= 0.95 * tiles[1])


@pytest.mark.parametrize("grid,window,batch,n,tau", [
    ((20, 17, 1), (6, 5, 1), 1, 200, 7),       # partial edge windows
    ((9, 9, 6), (4, 4, 3), 2, 500, 10),        # 3D windows, two frames
    ((5, 5, 5), (5, 5, 5), 1, 125, 36),        # one completely full window
    ((12, 12, 1), (12, 12, 1), 1, 36, 36),     # N == tau exactly: no duplicates
    ((12, 12, 1), (12, 12, 1), 1, 1, 36),      # a single voxel
    ((300, 300, 1), (7, 9, 1), 1, 5000, 90),   # spans several sort tiles and a ragged tail
    ((64, 64, 8), (64, 64, 8), 1, 20000, 48),  # one huge window (20000 voxels -> 417 sets)
    ((64, 64, 1), (1, 1, 1), 1, 3000, 36),     # every voxel a window of its own: 128 one-row sets per tile
    ((64, 64, 1), (8, 8, 1), 1, 4096, 64),     # full windows of 64 voxels: every set has 64 rows, two fill a tile
    ((96, 96, 1), (6, 7, 1), 1, 9216, 42),     # full windows of 42 (36 at the edges): three sets per tile at most
])
def test_partition_bit_exact_small_and_edge_cases(gpu, oracle, grid, window, batch, n, tau):
    rng = np.random.default_rng(n + tau)
    _check_partition(gpu, oracle, di.unique_cells(rng, n, grid, batch), batch, grid, window, tau)


@pytest.mark.parametrize("grid,window,shift,batch,n,tau", [
    ((20, 17, 1), (6, 5, 1), (3, 2, 0), 1, 200, 7),
    ((9, 9, 6), (4, 4, 3), (2, 1, 1), 2, 500, 10),
    ((468, 468, 1), (24, 24, 1), (12, 12, 0), 1, 32000, 36),   # the hybrid partner of the 12 x 12 windows
    ((64, 64, 8), (12, 12, 8), (6, 6, 0), 1, 9000, 48),
])
def test_partition_shifted_bit_exact(gpu, oracle, grid, window, shift, batch, n, tau):
    """dsvt_partition_shifted (displaced window cut, hybrid window partition) against the oracle."""
    rng = np.random.default_rng(n + tau)
    if grid == (468, 468, 1):
        coords = di.make_config(2, with_feats=False)["coords"]  # the LiDAR-shaped frame of configuration 2
    else:
        coords = di.unique_cells(rng, n, grid, batch)
    nwin = batch * int(np.prod([-(-(g + s) // w) for g, w, s in zip(grid, window, shift)]))
    ctx = gpu.Context(n, nwin, 64)
    both = ctx.partition_rotated(dev(coords), batch, grid, window, tau, shift=shift)
    assert ctx.status_sync() == 0
    for axis in (0, 1):
        ref = oracle.partition(coords, batch, grid, window, tau, axis, shift=shift)
        _compare_table(both[axis], ref, n, axis, extras=False)
    with pytest.raises(gpu.DsvtError):
        ctx.partition_rotated(dev(coords), batch, grid, window, tau, shift=(window[0], 0, 0))


def test_hybrid_window_backbone_matches_oracle(gpu, oracle):
    """Four blocks that alternate 12 x 12 windows with 24 x 24 windows displaced by (12, 12) (hybrid window
    partition, Sec. 3.2), whole small frame, bf16 weights: pipeline.Stage against the oracle block by block."""
    from paper_2301_06051_b200 import pipeline

    cfg = di.random_case(21, 3000, (96, 96, 1), (12, 12, 1), 36, 192, 8, hidden=384, layernorm=True, bf16=True,
                         n_blocks=4)
    specs = [((12, 12, 1), None), ((24, 24, 1), (12, 12, 0))] * 2
    nwin = int(np.prod([-(-(96 + 12) // 12)] * 2))
    ctx = gpu.Context(cfg["n"], nwin, 192)
    stage = pipeline.Stage(ctx, cfg["blocks"], 1, cfg["grid"], cfg["window"], 36, gpu.BF16_FP32ACC, cfg["n"],
                           block_windows=specs)
    x = dev(cfg["feats"])
    y = torch.empty_like(x)
    stage.forward(dev(cfg["coords"]), x, y)
    assert ctx.status_sync() == 0
    want = cfg["feats"].astype(np.float64)
    for blk, (window, shift) in zip(cfg["blocks"], specs):
        sh = shift or (0, 0, 0)
        t0 = oracle.partition(cfg["coords"], 1, cfg["grid"], window, 36, 0, shift=sh).set_table
        t1 = oracle.partition(cfg["coords"], 1, cfg["grid"], window, 36, 1, shift=sh).set_table
        want = oracle.block(want, t0, t1, blk)
    check_close(y.cpu().numpy(), want, "bf16", "hybrid-window backbone")


def test_partition_sorting_route_on_a_key_space_beyond_the_bitmap(gpu, oracle):
    """8400 x 8400 cells in 12 x 12 windows: 490000 windows x 160 padded cells exceed the context's
    64 Mi-key bitmap, so the call takes the radix-sort route; results are the same."""
    grid, window, n, tau = (8400, 8400, 1), (12, 12, 1), 6000, 36
    rng = np.random.default_rng(99)
    # clustered cells so that windows hold several voxels
    centre = rng.integers(100, 8300, size=(40, 2))
    pts = centre[rng.integers(0, 40, size=4 * n)] + rng.integers(-30, 31, size=(4 * n, 2))
    _, first = np.unique(pts[:, 0] * 8400 + pts[:, 1], return_index=True)
    pts = pts[np.sort(first)][:n]
    coords = np.zeros((pts.shape[0], 4), dtype=np.int32)
    coords[:, 1:3] = pts
    _check_partition(gpu, oracle, coords, 1, grid, window, tau)


def test_partition_flags_duplicate_cells_and_still_places_every_voxel(gpu):
    rng = np.random.default_rng(5)
    grid, window, tau = (24, 24, 1), (12, 12, 1), 5
    coords = di.unique_cells(rng, 200, grid, 1)
    coords = np.concatenate([coords, coords[:30], coords[:10]])  # 40 extra voxels in occupied cells
    n = coords.shape[0]
    ctx = gpu.Context(n, 4, 64)
    both = ctx.partition_rotated(dev(coords), 1, grid, window, tau)
    assert ctx.status_sync() & gpu.STATUS_DUPLICATE_CELL
    wid = (coords[:, 1] // 12) * 2 + coords[:, 2] // 12
    for t in both:
        tbl, ro = table_np(t)
        assert ro[-1] == n
        seen = np.zeros(n, dtype=np.int64)
        for row in tbl:
            u = np.unique(row)
            seen[u] += 1
            assert len(set(wid[u].tolist())) == 1
        assert np.all(seen == 1)


def test_partition_empty_and_errors(gpu):
    ctx = gpu.Context(100, 64, 64)
    empty = torch.zeros((0, 4), dtype=torch.int32, device="cuda")
    t = ctx.partition(empty, 1, (8, 8, 1), (4, 4, 1), 3, 0, extras=True)
    assert int(t.num_sets.item()) == 0 and int(t.win_start.sum().item()) == 0 and ctx.status_sync() == 0
    both = ctx.partition_rotated(empty, 1, (8, 8, 1), (4, 4, 1), 3)
    assert int(both[0].num_sets.item()) == 0 and int(both[1].num_sets.item()) == 0 and ctx.status_sync() == 0
    ok = dev(np.array([[0, 1, 1, 0], [0, 2, 2, 0], [0, 7, 7, 0]], dtype=np.int32))
    with pytest.raises(gpu.DsvtError):
        ctx.partition(ok, 1, (8, 8, 1), (4, 4, 1), 3, 2)  # bad axis
    with pytest.raises(gpu.DsvtError):
        ctx.partition(ok, 1, (800, 800, 1), (4, 4, 1), 3, 0)  # more windows than reserved
    # device-detected problems raise status bits instead of faulting
    bad = dev(np.array([[0, 1, 1, 0], [0, 9, 2, 0]], dtype=np.int32))
    ctx.partition(bad, 1, (8, 8, 1), (4, 4, 1), 3, 0)
    assert ctx.status_sync() & gpu.STATUS_BAD_COORD
    t = ctx.partition(ok, 1, (8, 8, 1), (4, 4, 1), 1, 0, cap_sets=2)  # three sets, room for two
    assert ctx.status_sync() & gpu.STATUS_TABLE_OVERFLOW
    assert int(t.num_sets.item()) == 2
    assert ctx.status_sync() == 0  # cleared by the read


# ------------------------------------------------------------------------------------------------
# set attention / layer / block
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("seed,n,grid,window,tau,C,heads,bf16", [
    (1, 150, (16, 16, 1), (6, 6, 1), 5, 16, 4, False),
    (2, 700, (30, 30, 4), (10, 10, 4), 36, 32, 8, False),
    (3, 90, (12, 12, 1), (12, 12, 1), 36, 64, 2, False),
    (4, 2500, (64, 64, 1), (12, 12, 1), 36, 128, 8, False),
    (5, 3000, (96, 96, 1), (30, 30, 1), 90, 128, 8, False),   # nuScenes-like window and set size
    (6, 1500, (48, 48, 1), (12, 12, 1), 36, 192, 8, True),
    (7, 1200, (48, 48, 2), (12, 12, 2), 48, 192, 8, True),
])
def test_set_attention_matches_oracle(gpu, oracle, seed, n, grid, window, tau, C, heads, bf16):
    cfg = di.random_case(seed, n, grid, window, tau, C, heads, bf16=bf16)
    L = cfg["blocks"][0][0]
    ctx = gpu.Context(n, _nwin(1, grid, window), C)
    w = gpu.device_weights(L, precision_of(cfg), ctx.device)
    x = dev(cfg["feats"])
    for axis in (0, 1):
        t = ctx.partition(dev(cfg["coords"]), 1, grid, window, tau, axis)
        out = torch.full_like(x, 123.0)
        ctx.set_attention(x, t, w, out)
        out2 = torch.full_like(x, 321.0)
        ctx.set_attention(x, t, w, out2, use_rowoff=False)  # row offsets derived from the table
        assert ctx.status_sync() == 0
        ref_t = oracle.partition(cfg["coords"], 1, grid, window, tau, axis).set_table
        want, covered = oracle.set_attention(cfg["feats"], ref_t, L["W_qkv"], L["b_qkv"], L["W_o"], L["b_o"], heads)
        assert covered.all()
        check_close(out.cpu().numpy(), want, cfg["precision"], "set_attention axis %d" % axis)
        if bf16:  # the tensor-core kernel: a tile plan made without the windows puts the sets into other tiles, and
            # a set's place in its tile decides how its attention is blocked: same result up to rounding
            check_close(out2.cpu().numpy(), want, cfg["precision"], "set_attention axis %d, derived offsets" % axis)
            assert float((out - out2).abs().max()) <= 1e-2 * float(np.abs(want).max())
        else:
            assert torch.equal(out, out2)


def test_set_attention_arbitrary_table_positional_term_and_untouched_rows(gpu, oracle):
    """A caller-made table (not from dsvt_partition): partial sets, duplicates in odd places,
    voxels in no set, table capacity larger than the set count, no biases."""
    rng = np.random.default_rng(5)
    n, C, heads, tau = 60, 32, 4, 6
    L = di.make_layer(rng, C, heads, 0, False, False)
    x = rng.standard_normal((n, C), dtype=np.float32)
    pe = rng.standard_normal((n, C), dtype=np.float32)
    table = np.array([[3, 3, 3, 7, 9, 9], [10, 11, 12, 13, 14, 15], [20, 20, 20, 20, 20, 20], [30, 31, 31, 32, 32, 33],
                      [59, 58, 57, 56, 55, 54], [40, 41, 41, 41, 42, 42]], dtype=np.int32)
    ctx = gpu.Context(n, 8, C)
    w = gpu.device_weights(L, gpu.FP32, ctx.device)
    w["b_qkv"] = None
    w["b_o"] = None
    for with_rowoff in (True, False):
        t = upload_table(table, with_rowoff=with_rowoff, cap_extra=5)
        out = torch.full((n, C), 55.0, device="cuda")
        ctx.set_attention(dev(x), t, w, out, pe=dev(pe))
        assert ctx.status_sync() == 0
        want = np.full((n, C), 55.0)
        want, covered = oracle.set_attention(x, table, L["W_qkv"], None, L["W_o"], None, heads, pe=pe, out=want)
        assert covered.sum() == 23
        check_close(out.cpu().numpy(), want, "fp32", "arbitrary table")
        assert np.all(out.cpu().numpy()[covered == 0] == 55.0)
    # an index outside [0, n) is skipped and flagged, never dereferenced
    bad = table.copy()
    bad[1, 2] = n + 5
    out = torch.zeros((n, C), device="cuda")
    ctx.set_attention(dev(x), upload_table(bad), w, out)
    assert ctx.status_sync() & gpu.STATUS_BAD_INDEX


def test_empty_inputs_are_no_ops(gpu):
    ctx = gpu.Context(16, 4, 32)
    rng = np.random.default_rng(1)
    L = di.make_layer(rng, 32, 4, 64, True, False)
    w = gpu.device_weights(L, gpu.FP32, ctx.device)
    x = torch.zeros((0, 32), device="cuda")
    t = upload_table(np.zeros((0, 6), dtype=np.int32))
    ctx.layer(x, t, w, x)
    ctx.set_attention(x, t, w, torch.zeros((0, 32), device="cuda"))
    assert ctx.status_sync() == 0


def _run_blocks_gpu(gpu, cfg, blocks, coords, feats, ctx=None):
    from paper_2301_06051_b200 import pipeline

    n = coords.shape[0]
    ctx = ctx or gpu.Context(n, _nwin(cfg["batch"], cfg["grid"], cfg["window"]), cfg["C"])
    st = pipeline.Stage(ctx, blocks, cfg["batch"], cfg["grid"], cfg["window"], cfg["set_size"], precision_of(cfg), n)
    x = dev(feats)
    y = torch.empty_like(x)
    st.forward(dev(coords), x, y)
    assert ctx.status_sync() == 0
    return y.cpu().numpy()


def _run_blocks_oracle(oracle, cfg, blocks, coords, feats):
    p0 = oracle.partition(coords, cfg["batch"], cfg["grid"], cfg["window"], cfg["set_size"], 0)
    p1 = oracle.partition(coords, cfg["batch"], cfg["grid"], cfg["window"], cfg["set_size"], 1)
    x = feats.astype(np.float64)
    for blk in blocks:
        x = oracle.block(x, p0.set_table, p1.set_table, blk)
    return x


def test_config1_block_fp32(gpu, oracle):
    """Config 1: 2000 pillars on 64x64, C = 128, one block of two attention layers, fp32 throughout."""
    cfg = di.make_config(1)
    got = _run_blocks_gpu(gpu, cfg, cfg["blocks"], cfg["coords"], cfg["feats"])
    want = _run_blocks_oracle(oracle, cfg, cfg["blocks"], cfg["coords"], cfg["feats"])
    check_close(got, want, "fp32", "config 1 block")


@pytest.mark.parametrize("bf16", [False, True])
def test_config1_shape_with_full_layers(gpu, oracle, bf16):
    """Config 1's frame with MLP and LayerNorm switched on, two blocks; also layer == block halves."""
    cfg = di.make_config(1)
    rng = np.random.default_rng(77)
    cfg["precision"] = "bf16" if bf16 else "fp32"
    blocks = [[di.make_layer(rng, 128, 8, 256, True, bf16) for _ in range(2)] for _ in range(2)]
    got = _run_blocks_gpu(gpu, cfg, blocks, cfg["coords"], cfg["feats"])
    want = _run_blocks_oracle(oracle, cfg, blocks, cfg["coords"], cfg["feats"])
    check_close(got, want, cfg["precision"], "config 1 frame, full layers")
    # dsvt_layer on its own, not in place, equals the oracle layer
    ctx = gpu.Context(cfg["n"], 36, 128)
    t0 = ctx.partition(dev(cfg["coords"]), 1, cfg["grid"], cfg["window"], 36, 0)
    w = gpu.device_weights(blocks[0][0], precision_of(cfg), ctx.device)
    y = torch.empty((cfg["n"], 128), device="cuda")
    ctx.layer(dev(cfg["feats"]), t0, w, y)
    ref_t = oracle.partition(cfg["coords"], 1, cfg["grid"], cfg["window"], 36, 0).set_table
    check_close(y.cpu().numpy(), oracle.layer(cfg["feats"], ref_t, blocks[0][0]), cfg["precision"], "layer")


def _sample_windows(oracle, cfg, coords, n_target, seed, win=None):
    """Voxel indices of randomly chosen whole windows holding about n_target voxels."""
    win = win or cfg["window"]
    p = oracle.partition(coords, cfg["batch"], cfg["grid"], win, cfg["set_size"], 0)
    rng = np.random.default_rng(seed)
    order = rng.permutation(np.flatnonzero(p.win_count > 0))
    # always include the fullest and the emptiest windows
    # always include the fullest window and the first and last non-empty ones (the first and the last tiles)
    nonempty = np.flatnonzero(p.win_count > 0)
    order = np.concatenate([[np.argmax(p.win_count), nonempty[0], nonempty[-1]], order])
    sel, total = [], 0
    for w in order:
        sel.append(p.perm[p.win_start[w]:p.win_start[w + 1]])
        total += sel[-1].shape[0]
        if total >= n_target:
            break
    return np.sort(np.unique(np.concatenate(sel)))


@pytest.mark.parametrize("cid,n_sample", [(2, 2500), (3, 2500), (4, 2500), (6, 2500)])
def test_backbone_full_size_bf16_on_sampled_windows(gpu, oracle, cid, n_sample):
    """Configs 2-4 (and the nuScenes-shaped extra, 6: windows 30 x 30, set size 90, C=128) at full size (four
    blocks, bf16 weights).  The backbone is window-local (both
    layers of every block use the same windows), so the oracle recomputes whole sampled windows."""
    cfg = di.make_config(cid)
    got = _run_blocks_gpu(gpu, cfg, cfg["blocks"], cfg["coords"], cfg["feats"])
    assert np.all(np.isfinite(got))
    sel = _sample_windows(oracle, cfg, cfg["coords"], n_sample, cid)
    want = _run_blocks_oracle(oracle, cfg, cfg["blocks"], cfg["coords"][sel], cfg["feats"][sel])
    check_close(got[sel], want, "bf16", "config %d backbone, %d sampled voxels" % (cid, sel.shape[0]))
    # one block on its own as well (per-block error, not only end to end)
    got1 = _run_blocks_gpu(gpu, cfg, cfg["blocks"][:1], cfg["coords"], cfg["feats"])
    want1 = _run_blocks_oracle(oracle, cfg, cfg["blocks"][:1], cfg["coords"][sel], cfg["feats"][sel])
    check_close(got1[sel], want1, "bf16", "config %d first block" % cid)


@pytest.mark.parametrize("cid", [2, 6])
def test_backbone_whole_frame_against_the_oracle(gpu, oracle, cid):
    """Configurations 2 and 6 (the nuScenes-shaped extra) in full: every voxel of the frame through all four
    blocks against the oracle, not a sample.  Prints the per-row relative error beside the tensor-wide one."""
    cfg = di.make_config(cid)
    oracle.set_threads(oracle.max_threads())
    got = _run_blocks_gpu(gpu, cfg, cfg["blocks"], cfg["coords"], cfg["feats"])
    want = _run_blocks_oracle(oracle, cfg, cfg["blocks"], cfg["coords"], cfg["feats"])
    rel = check_close(got, want, "bf16", "config %d backbone, whole frame" % cid)
    print("config %d whole frame: tensor-wide relative error %.3e, largest per-row relative error %.3e"
          % (cid, rel, row_rel_error(got, want)))


def test_in_place_and_repeatability(gpu):
    cfg = di.make_config(2, n_override=6000)
    a = _run_blocks_gpu(gpu, cfg, cfg["blocks"][:2], cfg["coords"], cfg["feats"])
    b = _run_blocks_gpu(gpu, cfg, cfg["blocks"][:2], cfg["coords"], cfg["feats"])
    assert np.array_equal(a, b)  # no atomics on the float path: bitwise repeatable


@pytest.mark.parametrize("partition_ahead,lanes,depth", [(False, 1, 2), (True, 1, 2), (True, 2, 4), (True, 4, 8)])
def test_frame_stream_overlaps_copies_without_mixing_frames(gpu, partition_ahead, lanes, depth):
    """Seven different frames (different sizes and contents) through pipeline.FrameStream: plain, with the next
    frame's partition running ahead on its own stream, and with two compute lanes: every host output equals the
    frame's own device-resident run."""
    from paper_2301_06051_b200 import pipeline

    base = di.make_config(2, n_override=9000)
    n_max = 9000
    ctx = gpu.Context(n_max, _nwin(base["batch"], base["grid"], base["window"]), base["C"])
    st = pipeline.Stage(ctx, base["blocks"][:2], base["batch"], base["grid"], base["window"], base["set_size"],
                        precision_of(base), n_max)
    frames = []
    for k, n in enumerate([9000, 4000, 7000, 1, 8999, 2500, 6000]):
        rng = np.random.default_rng(100 + k)
        coords = di.unique_cells(rng, n, base["grid"], base["batch"])
        feats = rng.standard_normal((n, base["C"]), dtype=np.float32)
        frames.append((torch.from_numpy(coords).pin_memory(), torch.from_numpy(feats).pin_memory(),
                       torch.full((n, base["C"]), 5.0).pin_memory()))
    fs = pipeline.FrameStream(st, n_max, base["C"], depth=depth, partition_ahead=partition_ahead, lanes=lanes)
    for c, f, o in frames:
        fs.submit(c, f, o)
    fs.wait()
    assert fs.status_sync() == 0
    for c, f, o in frames:
        y = torch.empty((f.shape[0], base["C"]), device="cuda")
        st.forward(c.cuda(), f.cuda(), y)
        assert torch.equal(y.cpu(), o)


def test_layer_cta_cap_keeps_results_and_rejects_negative_values(gpu):
    """dsvt_set_layer_ctas: a block on 7 CTAs (dozens of tiles each) is bitwise the block on one CTA per SM."""
    cfg = di.make_config(2, n_override=20000)
    n, C = cfg["n"], cfg["C"]
    ctx = gpu.Context(n, _nwin(cfg["batch"], cfg["grid"], cfg["window"]), C)
    coords, x = dev(cfg["coords"]), dev(cfg["feats"])
    t0, t1 = ctx.partition_rotated(coords, cfg["batch"], cfg["grid"], cfg["window"], cfg["set_size"])
    w = [gpu.device_weights(l, precision_of(cfg), ctx.device) for l in cfg["blocks"][0]]
    full, capped = torch.empty_like(x), torch.empty_like(x)
    ctx.block(x, t0, t1, w, full)
    ctx.set_layer_ctas(7)
    ctx.block(x, t0, t1, w, capped)
    ctx.set_layer_ctas(0)
    assert ctx.status_sync() == 0
    assert torch.equal(full, capped)
    with pytest.raises(gpu.DsvtError):
        ctx.set_layer_ctas(-1)


def test_frame_stream_resident_frames_on_two_lanes(gpu):
    """Ten device-resident frames (four rotating buffer sets, different sizes and contents) through the two-lane
    pipeline with the partition running ahead: every output equals the frame's own single-stream run."""
    from paper_2301_06051_b200 import pipeline

    base = di.make_config(2, n_override=8000)
    n_max = 8000
    ctx = gpu.Context(n_max, _nwin(base["batch"], base["grid"], base["window"]), base["C"])
    st = pipeline.Stage(ctx, base["blocks"][:2], base["batch"], base["grid"], base["window"], base["set_size"],
                        precision_of(base), n_max)
    fs = pipeline.FrameStream(st, n_max, base["C"], depth=4, lanes=2, layer_ctas=20)  # several tiles per CTA
    sizes = [8000, 3000, 1, 7999, 5000, 6500, 2, 4000, 8000, 1000]
    bufs = [(torch.empty((n_max, 4), dtype=torch.int32, device="cuda"), torch.empty((n_max, base["C"]), device="cuda"),
             torch.empty((n_max, base["C"]), device="cuda")) for _ in range(4)]
    want, got = [], []
    for k, n in enumerate(sizes):
        rng = np.random.default_rng(500 + k)
        c = torch.from_numpy(di.unique_cells(rng, n, base["grid"], base["batch"])).cuda()
        f = torch.from_numpy(rng.standard_normal((n, base["C"]), dtype=np.float32)).cuda()
        y = torch.empty_like(f)
        st.forward(c, f, y)
        want.append(y.cpu())
        torch.cuda.synchronize()
        if k >= 4:  # the set is handed in again: its previous frame's result must have been read first
            fs.join(torch.cuda.current_stream())
            got.append(bufs[k % 4][2][: sizes[k - 4]].cpu())
        cb, xb, yb = bufs[k % 4]
        cb[:n].copy_(c); xb[:n].copy_(f)
        torch.cuda.synchronize()
        fs.submit_resident(cb[:n], xb[:n], yb[:n])
    fs.wait()
    for k in range(len(sizes) - 4, len(sizes)):
        got.append(bufs[k % 4][2][: sizes[k]].cpu())
    assert fs.status_sync() == 0
    for k, (g, w) in enumerate(zip(got, want)):
        assert torch.equal(g, w), "frame %d" % k


# ------------------------------------------------------------------------------------------------
# pooling
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("mask_empty", [0, 1])
@pytest.mark.parametrize("grid,pool,batch,n,C,heads,with_pe,bf16", [
    ((16, 16, 1), (2, 2, 1), 1, 120, 16, 4, False, False),
    ((9, 7, 8), (2, 2, 2), 2, 400, 32, 4, True, False),
    ((6, 6, 8), (1, 1, 4), 1, 150, 32, 8, False, False),
    ((40, 40, 1), (3, 3, 1), 1, 900, 64, 8, True, False),
    ((100, 100, 1), (2, 2, 1), 1, 4000, 192, 8, False, True),
    ((20, 20, 16), (2, 2, 4), 1, 3000, 192, 8, True, True),
    ((60, 60, 1), (2, 2, 1), 2, 5000, 128, 8, True, True),     # several tiles per CTA, ragged last tile
    ((30, 30, 4), (3, 3, 2), 1, 2500, 64, 4, False, True),      # 18 slots per region
    ((50, 50, 1), (2, 1, 1), 1, 2000, 128, 4, False, True),     # 2 slots: 64 regions per tile
    ((36, 36, 2), (2, 2, 2), 1, 1500, 64, 8, True, True),       # head dim 8
    ((40, 40, 1), (2, 2, 1), 1, 1200, 192, 4, True, True),      # head dim 48
    ((260, 260, 1), (2, 2, 1), 1, 45000, 64, 4, False, True),   # more tiles than SMs: several tiles per CTA
])
def test_pool_matches_oracle(gpu, oracle, grid, pool, batch, n, C, heads, with_pe, bf16, mask_empty):
    rng = np.random.default_rng(n + C)
    coords = di.unique_cells(rng, n, grid, batch)
    feats = rng.standard_normal((n, C), dtype=np.float32)
    nslots = pool[0] * pool[1] * pool[2]
    Wt = di.make_pool_weights(rng, C, heads, bf16, nslots, with_pe)
    regions = batch * int(np.prod([-(-g // p) for g, p in zip(grid, pool)]))
    ctx = gpu.Context(n, regions, C)
    w = gpu.device_weights(Wt, gpu.BF16_FP32ACC if bf16 else gpu.FP32, ctx.device)
    oc, of, num, reg, slot = ctx.pool(dev(coords), dev(feats), batch, grid, pool, w, mask_empty=mask_empty, extras=True)
    assert ctx.status_sync() == 0
    ref = oracle.pool(coords, feats, batch, grid, pool, Wt["W_q"], Wt["W_k"], Wt["W_v"], Wt["W_o"], Wt["b_q"],
                      Wt["b_k"], Wt["b_v"], Wt["b_o"], heads, slot_pe=Wt["slot_pe"], mask_empty=mask_empty)
    m = int(num.item())
    assert m == ref.coords.shape[0]
    assert np.array_equal(oc[:m].cpu().numpy(), ref.coords)
    assert np.array_equal(reg.cpu().numpy(), ref.region_of)
    assert np.array_equal(slot.cpu().numpy(), ref.slot_of)
    check_close(of[:m].cpu().numpy(), ref.feats, "bf16" if bf16 else "fp32", "pool")


def test_pool_flags_duplicate_cells_and_overflow(gpu):
    rng = np.random.default_rng(3)
    C = 16
    Wt = di.make_pool_weights(rng, C, 4, False)
    ctx = gpu.Context(16, 64, C)
    w = gpu.device_weights(Wt, gpu.FP32, ctx.device)
    coords = np.array([[0, 1, 1, 0], [0, 1, 1, 0], [0, 5, 5, 0]], dtype=np.int32)
    feats = rng.standard_normal((3, C), dtype=np.float32)
    ctx.pool(dev(coords), dev(feats), 1, (8, 8, 1), (2, 2, 1), w)
    assert ctx.status_sync() & gpu.STATUS_DUPLICATE_CELL
    coords = np.array([[0, 1, 1, 0], [0, 3, 1, 0], [0, 5, 5, 0]], dtype=np.int32)
    oc, of, num, _, _ = ctx.pool(dev(coords), dev(feats), 1, (8, 8, 1), (2, 2, 1), w, cap_m=2)
    assert ctx.status_sync() & gpu.STATUS_TABLE_OVERFLOW
    assert int(num.item()) == 2


def test_config5_blocks_pool_blocks_on_sampled_windows(gpu, oracle):
    """Config 5 at full size: two blocks, 2x2x1 attention pooling, two blocks at half resolution.
    A 12x12 window of the pooled grid covers a 24x24 area of the input grid, i.e. four whole input
    windows, so the chain is local to such areas and the oracle recomputes sampled areas."""
    from paper_2301_06051_b200 import pipeline

    cfg = di.make_config(5)
    bb = pipeline.Backbone(cfg)
    x = dev(cfg["feats"])
    oc, of, num = bb.forward(dev(cfg["coords"]), x, torch.empty_like(x))
    assert bb.ctx.status_sync() == 0
    oc, of = oc.cpu().numpy(), of.cpu().numpy()
    assert np.all(np.isfinite(of))
    coords = cfg["coords"]
    sel = _sample_windows(oracle, cfg, coords, 3000, 5, win=(24, 24, 1))
    cs, fs = coords[sel], cfg["feats"][sel]
    mid = _run_blocks_oracle(oracle, cfg, cfg["blocks"], cs, fs)
    pw = cfg["pool"]
    pooled = oracle.pool(cs, mid, 1, cfg["grid"], cfg["pool_shape"], pw["W_q"], pw["W_k"], pw["W_v"], pw["W_o"],
                         pw["b_q"], pw["b_k"], pw["b_v"], pw["b_o"], cfg["heads"])
    cfg2 = dict(cfg, grid=(468, 468, 1))
    want = _run_blocks_oracle(oracle, cfg2, cfg["blocks_after_pool"], pooled.coords, pooled.feats)
    # match rows by pooled coordinate
    key = lambda c: (c[:, 1].astype(np.int64) * 468 + c[:, 2])
    pos = {k: i for i, k in enumerate(key(oc).tolist())}
    rows = np.array([pos[k] for k in key(pooled.coords).tolist()])
    assert np.all(np.diff(key(oc)) > 0)  # ascending pooled coordinates
    check_close(of[rows], want, "bf16", "config 5 chain, %d pooled voxels" % rows.shape[0])


def test_dsvt_v_stage_layout_on_sampled_windows(gpu, oracle):
    """The voxel variant's layout at full size (configuration 7: four one-block stages, z windows 32 / 8 / 2 / 1,
    pooling along z by 4, 4, 2, set size 48).  Pooling along z keeps the 12 x 12 footprint of a window, so the whole
    chain is local to a footprint and the oracle recomputes sampled footprints."""
    from paper_2301_06051_b200 import pipeline

    cfg = di.make_config(7)
    bb = pipeline.StagedBackbone(cfg)
    oc, of = bb.forward(dev(cfg["coords"]), dev(cfg["feats"]))
    assert bb.ctx.status_sync() == 0
    oc, of = oc.cpu().numpy(), of.cpu().numpy()
    assert np.all(np.isfinite(of))
    sel = _sample_windows(oracle, cfg, cfg["coords"], 2500, 7)
    cs, fs = cfg["coords"][sel], cfg["feats"][sel].astype(np.float64)
    grid = tuple(cfg["grid"])
    for i, st in enumerate(cfg["stages"]):
        c_i = dict(cfg, grid=grid, window=st["window"])
        fs = _run_blocks_oracle(oracle, c_i, st["blocks"], cs, fs)
        if i < len(cfg["pools"]):
            pl = cfg["pools"][i]
            pw = pl["weights"]
            pooled = oracle.pool(cs, fs, 1, grid, pl["shape"], pw["W_q"], pw["W_k"], pw["W_v"], pw["W_o"],
                                 pw["b_q"], pw["b_k"], pw["b_v"], pw["b_o"], cfg["heads"])
            cs, fs = pooled.coords, pooled.feats
            grid = tuple(-(-grid[a] // pl["shape"][a]) for a in range(3))
    assert grid == (468, 468, 1)
    key = lambda c: (c[:, 1].astype(np.int64) * 468 + c[:, 2])
    assert np.all(np.diff(key(oc)) > 0)  # ascending pooled coordinates
    pos = {k: i for i, k in enumerate(key(oc).tolist())}
    rows = np.array([pos[k] for k in key(cs).tolist()])
    check_close(of[rows], fs, "bf16", "DSVT-V stage layout, %d output voxels" % rows.shape[0])


def test_counts_that_live_on_the_device(gpu, oracle):
    """dsvt_partition_counted and dsvt_pool_counted: the voxel count is read on the device, the arrays have the
    capacity's length and garbage past the count.  The tables are bit-exact those of the oracle for the counted
    voxels; the pooling equals dsvt_pool on the truncated arrays; a count of zero gives empty results."""
    rng = np.random.default_rng(5)
    grid, window, tau, n, k = (60, 60, 2), (12, 12, 2), 36, 3000, 1777
    coords = di.unique_cells(rng, n, grid, 1)
    junk = coords.copy()
    junk[k:] = 10 ** 6  # (would raise the bad-coordinate bit if it were read)
    ctx = gpu.Context(n, _nwin(1, grid, window), 64)
    cnt = dev(np.array([k], dtype=np.int32))
    both = ctx.partition_rotated(dev(junk), 1, grid, window, tau, n_dev=cnt)
    assert ctx.status_sync() == 0
    for axis in (0, 1):
        _compare_table(both[axis], oracle.partition(coords[:k], 1, grid, window, tau, axis), k, axis, extras=False)
    zero = dev(np.array([0], dtype=np.int32))
    both = ctx.partition_rotated(dev(junk), 1, grid, window, tau, n_dev=zero)
    assert ctx.status_sync() == 0 and int(both[0].num_sets.item()) == 0 and int(both[1].num_sets.item()) == 0
    assert int(both[0].set_rowoff[0].item()) == 0 and int(both[0].set_rowoff[both[0].cap_sets + 1].item()) == 0
    # pooling
    C, heads = 64, 4
    feats = rng.standard_normal((n, C), dtype=np.float32)
    w = gpu.device_weights(di.make_pool_weights(rng, C, heads, True), gpu.BF16_FP32ACC, ctx.device)
    ctx2 = gpu.Context(n, 30 * 30 * 2, C)
    oc, of, num, _, _ = ctx2.pool(dev(junk), dev(feats), 1, grid, (2, 2, 1), w, n_dev=cnt)
    rc, rf, rnum, _, _ = ctx2.pool(dev(coords[:k]), dev(feats[:k]), 1, grid, (2, 2, 1), w)
    assert ctx2.status_sync() == 0
    m = int(rnum.item())
    assert int(num.item()) == m and torch.equal(oc[:m], rc[:m]) and torch.equal(of[:m], rf[:m])
    oc, of, num, _, _ = ctx2.pool(dev(junk), dev(feats), 1, grid, (2, 2, 1), w, n_dev=zero)
    assert ctx2.status_sync() == 0 and int(num.item()) == 0


def test_layers_beyond_the_tile_plan_capacity(gpu, oracle):
    """More sets than the partition's tile plan covers (set size 4: 30,000 sets): the plan entry says "no plan" and the
    layer kernel cuts its tiles by row ranges.  One block at full size against the oracle on sampled windows."""
    cfg = di.random_case(21, 110000, (400, 400, 1), (12, 12, 1), 4, 64, 4, hidden=128, layernorm=True, bf16=True)
    ctx = gpu.Context(cfg["n"], _nwin(1, cfg["grid"], cfg["window"]), 64)
    t0, t1 = ctx.partition_rotated(dev(cfg["coords"]), 1, cfg["grid"], cfg["window"], 4)
    S = int(t0.num_sets.item())
    assert S > 24576 and int(t0.set_rowoff[t0.cap_sets + 1].item()) == -1
    got = _run_blocks_gpu(gpu, cfg, cfg["blocks"], cfg["coords"], cfg["feats"], ctx=ctx)
    assert np.all(np.isfinite(got))
    sel = _sample_windows(oracle, cfg, cfg["coords"], 2500, 3)
    want = _run_blocks_oracle(oracle, cfg, cfg["blocks"], cfg["coords"][sel], cfg["feats"][sel])
    check_close(got[sel], want, "bf16", "one block, %d sets without a plan" % S)
