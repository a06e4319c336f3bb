"""GPU parity through the C ABI: relative position bias on the attention logits, and the BEV projection."""
import numpy as np
import pytest
import torch

import dsvt_inputs as di
from gpu_helpers import check_close, dev, precision_of, upload_table

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gpu():
    from paper_2301_06051_b200 import api

    api.load()
    return api


def _nwin(batch, grid, window):
    return batch * int(np.prod([-(-g // w) for g, w in zip(grid, window)]))


def _with_bias(rng, layer, heads, extent, oracle):
    L = dict(layer)
    L["rpb"] = rng.standard_normal((heads, oracle.rel_bias_len(extent))).astype(np.float32)
    L["rpb_extent"] = tuple(extent)
    return L


@pytest.mark.parametrize("seed,n,grid,window,tau,C,heads,bf16", [
    (31, 150, (16, 16, 1), (6, 6, 1), 5, 16, 4, False),
    (32, 700, (30, 30, 4), (10, 10, 4), 36, 32, 8, False),
    (33, 2500, (64, 64, 1), (12, 12, 1), 36, 128, 8, False),
    (34, 3000, (96, 96, 1), (30, 30, 1), 90, 128, 8, False),
    (35, 1500, (48, 48, 1), (12, 12, 1), 36, 192, 8, True),
    (36, 1200, (48, 48, 2), (12, 12, 2), 48, 192, 8, True),
    (37, 3000, (96, 96, 1), (30, 30, 1), 90, 128, 8, True),    # one attention item per set (set size above 48)
    (38, 2000, (60, 60, 1), (12, 12, 1), 36, 128, 4, True),    # head dimension 32
    (39, 900, (24, 24, 40), (12, 12, 32), 36, 64, 4, True),    # 33,327 entries: offsets use 16 of the 16 index bits
    (40, 900, (24, 24, 40), (12, 12, 40), 36, 64, 4, True),    # 41,791 entries per head
    (43, 900, (32, 32, 40), (16, 16, 36), 36, 64, 4, True),    # 68,231 entries: beyond 16-bit differences (FMA kernel)
])
def test_set_attention_with_relative_position_bias(gpu, oracle, seed, n, grid, window, tau, C, heads, bf16):
    cfg = di.random_case(seed, n, grid, window, tau, C, heads, bf16=bf16)
    L = _with_bias(np.random.default_rng(seed), cfg["blocks"][0][0], heads, window, oracle)
    ctx = gpu.Context(n, _nwin(1, grid, window), C)
    w = gpu.device_weights(L, precision_of(cfg), ctx.device)
    x, coords = dev(cfg["feats"]), dev(cfg["coords"])
    for axis in (0, 1):
        t = ctx.partition(coords, 1, grid, window, tau, axis)
        out = torch.full_like(x, 9.0)
        ctx.set_attention(x, t, w, out, coords=coords)
        assert ctx.status_sync() == 0
        ref_t = oracle.partition(cfg["coords"], 1, grid, window, tau, axis).set_table
        want, covered = oracle.set_attention(cfg["feats"], ref_t, L["W_qkv"], L["b_qkv"], L["W_o"], L["b_o"], heads,
                                             rpb=L["rpb"], coords=cfg["coords"], rpb_extent=window)
        assert covered.all()
        check_close(out.cpu().numpy(), want, cfg["precision"], "biased set attention axis %d" % axis)
        plain, _ = oracle.set_attention(cfg["feats"], ref_t, L["W_qkv"], L["b_qkv"], L["W_o"], L["b_o"], heads)
        assert np.abs(plain - want).max() > 1e-2  # the case would notice a dropped bias


@pytest.mark.parametrize("bf16", [False, True])
def test_block_with_relative_position_bias_and_a_larger_table(gpu, oracle, bf16):
    """Two full layers (MLP, LayerNorm) with per-layer bias tables cut for a window larger than the partition's."""
    seed, n, grid, window, tau, C, heads = 41, 1800, (60, 60, 1), (12, 12, 1), 36, 64, 4
    cfg = di.random_case(seed, n, grid, window, tau, C, heads, hidden=128, layernorm=True, bf16=bf16)
    rng = np.random.default_rng(seed)
    extent = (14, 13, 2)
    layers = [_with_bias(rng, l, heads, extent, oracle) for l in cfg["blocks"][0]]
    ctx = gpu.Context(n, _nwin(1, grid, window), C)
    ws = [gpu.device_weights(l, precision_of(cfg), ctx.device) for l in layers]
    x, coords = dev(cfg["feats"]), dev(cfg["coords"])
    t0, t1 = ctx.partition_rotated(coords, 1, grid, window, tau)
    y = torch.empty_like(x)
    ctx.block(x, t0, t1, ws, y, coords=coords)
    assert ctx.status_sync() == 0
    p0 = oracle.partition(cfg["coords"], 1, grid, window, tau, 0).set_table
    p1 = oracle.partition(cfg["coords"], 1, grid, window, tau, 1).set_table
    want = oracle.block(cfg["feats"], p0, p1, layers, coords=cfg["coords"])
    check_close(y.cpu().numpy(), want, cfg["precision"], "biased block")
    # dsvt_layer alone
    y1 = torch.empty_like(x)
    ctx.layer(x, t0, ws[0], y1, coords=coords)
    check_close(y1.cpu().numpy(), oracle.layer(cfg["feats"], p0, layers[0], coords=cfg["coords"]), cfg["precision"],
                "biased layer")


def test_long_bias_table_runs_on_the_tensor_core_kernel(gpu, oracle):
    """A table of 33,327 entries per head (window 12 x 12 x 32): row indices are kept modulo 2^16, every offset of a
    covered set still fits.  Two bf16 layers with such tables go out as one launch (the chained tensor-core kernel;
    the FMA kernel would take one launch per layer) and match the oracle."""
    seed, n, grid, window, tau, C, heads = 42, 2500, (36, 36, 40), (12, 12, 32), 36, 192, 8
    cfg = di.random_case(seed, n, grid, window, tau, C, heads, hidden=384, layernorm=True, bf16=True)
    rng = np.random.default_rng(seed)
    layers = [_with_bias(rng, l, heads, window, oracle) for l in cfg["blocks"][0]]
    ctx = gpu.Context(n, _nwin(1, grid, window), C)
    ws = [gpu.device_weights(l, precision_of(cfg), ctx.device) for l in layers]
    x, coords = dev(cfg["feats"]), dev(cfg["coords"])
    t0, t1 = ctx.partition_rotated(coords, 1, grid, window, tau)
    y = torch.empty_like(x)
    before = ctx.launch_count()
    ctx.block(x, t0, t1, ws, y, coords=coords)
    assert ctx.launch_count() - before == 1
    assert ctx.status_sync() == 0
    p0 = oracle.partition(cfg["coords"], 1, grid, window, tau, 0).set_table
    p1 = oracle.partition(cfg["coords"], 1, grid, window, tau, 1).set_table
    want = oracle.block(cfg["feats"], p0, p1, layers, coords=cfg["coords"])
    check_close(y.cpu().numpy(), want, cfg["precision"], "block with long bias tables")
    plain = oracle.block(cfg["feats"], p0, p1, cfg["blocks"][0])
    assert np.abs(plain - want).max() > 1e-2


def test_bias_table_narrower_than_a_set_is_flagged(gpu, oracle):
    rng = np.random.default_rng(3)
    n, C, heads, tau = 40, 16, 4, 4
    L = _with_bias(rng, di.make_layer(rng, C, heads, 0, False, False), heads, (3, 3, 1), oracle)
    coords = np.zeros((n, 4), dtype=np.int32)
    coords[:, 1] = np.arange(n) % 8
    coords[:, 2] = np.arange(n) // 8
    ctx = gpu.Context(n, 8, C)
    w = gpu.device_weights(L, gpu.FP32, ctx.device)
    x = dev(rng.standard_normal((n, C), dtype=np.float32))
    ok = np.array([[0, 1, 2, 2], [8, 9, 10, 10]], dtype=np.int32)       # spread 3 cells along x: covered
    out = torch.zeros((n, C), device="cuda")
    ctx.set_attention(x, upload_table(ok), w, out, coords=dev(coords))
    assert ctx.status_sync() == 0
    wide = np.array([[0, 1, 2, 3], [8, 9, 10, 10]], dtype=np.int32)     # spread 4 cells: not covered by L = 3
    ctx.set_attention(x, upload_table(wide), w, out, coords=dev(coords))
    assert ctx.status_sync() & gpu.STATUS_BAD_INDEX
    assert torch.isfinite(out).all()
    # a bias without coordinates is refused on the host
    with pytest.raises(gpu.DsvtError):
        ctx.set_attention(x, upload_table(ok), w, out, coords=None)


@pytest.mark.parametrize("cid", [2, 6])
def test_full_size_frame_with_bias_on_sampled_windows(gpu, oracle, cid):
    """One block of the full-size frame (bf16 weights, tensor-core kernel, several tiles per thread block) with a
    bias table per layer; whole sampled windows are recomputed by the oracle.  A table cut for a smaller window
    than the partition's is reported and harms nothing else."""
    cfg = di.make_config(cid)
    rng = np.random.default_rng(cid)
    heads, window, tau = cfg["heads"], cfg["window"], cfg["set_size"]
    layers = [_with_bias(rng, l, heads, window, oracle) for l in cfg["blocks"][0]]
    n = cfg["n"]
    ctx = gpu.Context(n, _nwin(cfg["batch"], cfg["grid"], window), cfg["C"])
    ws = [gpu.device_weights(l, gpu.BF16_FP32ACC, ctx.device) for l in layers]
    x, coords = dev(cfg["feats"]), dev(cfg["coords"])
    t0, t1 = ctx.partition_rotated(coords, cfg["batch"], cfg["grid"], window, tau)
    y = torch.empty_like(x)
    ctx.block(x, t0, t1, ws, y, coords=coords)
    assert ctx.status_sync() == 0
    got = y.cpu().numpy()
    assert np.all(np.isfinite(got))
    # whole windows holding about 2500 voxels
    p = oracle.partition(cfg["coords"], cfg["batch"], cfg["grid"], window, tau, 0)
    order = np.concatenate([[np.argmax(p.win_count)], rng.permutation(np.flatnonzero(p.win_count > 0))])
    sel, total = [], 0
    for w in order:
        sel.append(p.perm[p.win_start[w]:p.win_start[w + 1]])
        total += sel[-1].shape[0]
        if total >= 2500:
            break
    sel = np.sort(np.unique(np.concatenate(sel)))
    sc, sf = cfg["coords"][sel], cfg["feats"][sel]
    p0 = oracle.partition(sc, cfg["batch"], cfg["grid"], window, tau, 0).set_table
    p1 = oracle.partition(sc, cfg["batch"], cfg["grid"], window, tau, 1).set_table
    want = oracle.block(sf, p0, p1, layers, coords=sc)
    check_close(got[sel], want, "bf16", "config %d block with bias" % cid)
    plain = oracle.block(sf, p0, p1, cfg["blocks"][0])
    assert np.abs(plain - want).max() > 1e-2
    # too small a table: reported by the status word, results stay finite
    small = tuple(max(1, v // 2) for v in window)
    ws_small = [gpu.device_weights(_with_bias(rng, l, heads, small, oracle), gpu.BF16_FP32ACC, ctx.device)
                for l in cfg["blocks"][0]]
    ctx.block(x, t0, t1, ws_small, y, coords=coords)
    assert ctx.status_sync() & gpu.STATUS_BAD_INDEX
    assert torch.isfinite(y).all()


def test_bias_table_narrower_than_a_set_is_flagged_on_the_tensor_core_path(gpu, oracle):
    rng = np.random.default_rng(4)
    n, C, heads, tau = 40, 64, 4, 4
    L = _with_bias(rng, di.make_layer(rng, C, heads, 0, False, True), heads, (3, 3, 1), oracle)
    coords = np.zeros((n, 4), dtype=np.int32)
    coords[:, 1] = np.arange(n) % 8
    coords[:, 2] = np.arange(n) // 8
    ctx = gpu.Context(n, 8, C)
    w = gpu.device_weights(L, gpu.BF16_FP32ACC, ctx.device)
    xh = rng.standard_normal((n, C), dtype=np.float32)
    x = dev(xh)
    ok = np.array([[0, 1, 2, 2], [8, 9, 10, 10]], dtype=np.int32)
    out = torch.zeros((n, C), device="cuda")
    ctx.set_attention(x, upload_table(ok), w, out, coords=dev(coords))
    assert ctx.status_sync() == 0
    want, covered = oracle.set_attention(xh, ok, L["W_qkv"], L["b_qkv"], L["W_o"], L["b_o"], heads, rpb=L["rpb"],
                                         coords=coords, rpb_extent=(3, 3, 1))
    check_close(out.cpu().numpy()[covered == 1], want[covered == 1], "bf16", "caller-made table with bias")
    wide = np.array([[0, 1, 2, 3], [8, 9, 10, 10]], dtype=np.int32)
    ctx.set_attention(x, upload_table(wide), w, out, coords=dev(coords))
    assert ctx.status_sync() & gpu.STATUS_BAD_INDEX
    assert torch.isfinite(out).all()


# ------------------------------------------------------------------------------------------------ BEV projection
@pytest.mark.parametrize("grid,batch,n,C", [
    ((33, 7, 1), 1, 60, 8),       # one full 32-cell segment and a ragged tail of one cell
    ((100, 37, 1), 2, 1500, 64),
    ((20, 9, 4), 2, 500, 16),     # z cells stacked into channels
    ((5, 3, 2), 1, 0, 4),         # no voxels: a map of zeros
    ((64, 64, 1), 1, 4096, 192),  # every cell occupied
])
@pytest.mark.parametrize("channels_last", [False, True])
def test_bev_map_is_exact(gpu, oracle, grid, batch, n, C, channels_last):
    rng = np.random.default_rng(n + C)
    coords = di.unique_cells(rng, n, grid, batch)
    feats = rng.standard_normal((n, C), dtype=np.float32)
    ctx = gpu.Context(max(n, 1), 8, C)
    shape = (batch, grid[1], grid[0], C * grid[2]) if channels_last else (batch, C * grid[2], grid[1], grid[0])
    out = torch.full(shape, 7.0, device="cuda")  # stale contents must be overwritten
    ctx.bev_scatter(dev(coords.reshape(-1, 4)), dev(feats.reshape(-1, C)), batch, grid, channels_last, out=out)
    assert ctx.status_sync() == 0
    want = oracle.bev_scatter(coords, feats, batch, grid, channels_last)
    assert np.array_equal(out.cpu().numpy().astype(np.float64), want)


def test_bev_full_size_pillar_frame(gpu, oracle):
    cfg = di.make_config(2)
    ctx = gpu.Context(cfg["n"], 8, cfg["C"])
    out = ctx.bev_scatter(dev(cfg["coords"]), dev(cfg["feats"]), cfg["batch"], cfg["grid"])
    assert ctx.status_sync() == 0
    want = oracle.bev_scatter(cfg["coords"], cfg["feats"], cfg["batch"], cfg["grid"])
    assert np.array_equal(out.cpu().numpy(), want.astype(np.float32))


def test_bev_flags_bad_input(gpu):
    ctx = gpu.Context(8, 8, 8)
    feats = torch.ones((3, 8), device="cuda")
    dup = np.array([[0, 1, 1, 0], [0, 1, 1, 0], [0, 2, 2, 0]], dtype=np.int32)
    out = ctx.bev_scatter(dev(dup), feats, 1, (4, 4, 1))
    assert ctx.status_sync() & gpu.STATUS_DUPLICATE_CELL
    assert float(out.sum()) == 16.0  # two occupied cells of eight channels
    outside = np.array([[0, 1, 1, 0], [0, 4, 0, 0], [1, 0, 0, 0]], dtype=np.int32)
    out = ctx.bev_scatter(dev(outside), feats, 1, (4, 4, 1))
    assert ctx.status_sync() & gpu.STATUS_BAD_COORD
    assert float(out.sum()) == 8.0
    with pytest.raises(gpu.DsvtError):
        ctx.bev_scatter(dev(dup), torch.ones((3, 6), device="cuda"), 1, (4, 4, 1))  # C % 4 != 0
