"""dsvt_layers (a chain of layers in one launch) through the C ABI against the CPU oracle and against the same layers
launched one by one.  All tests need a B200."""
import numpy as np
import pytest
import torch

import dsvt_inputs as di
from gpu_helpers import check_close, dev, precision_of

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gpu():
    from paper_2301_06051_b200 import api

    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    api.load()
    return api


def _nwin(cfg):
    return cfg["batch"] * int(np.prod([-(-g // w) for g, w in zip(cfg["grid"], cfg["window"])]))


def _setup(gpu, cfg, blocks):
    ctx = gpu.Context(cfg["n"], _nwin(cfg), cfg["C"])
    t0, t1 = ctx.partition_rotated(dev(cfg["coords"]), cfg["batch"], cfg["grid"], cfg["window"], cfg["set_size"])
    ws = [gpu.device_weights(l, precision_of(cfg), ctx.device) for blk in blocks for l in blk]
    tabs = [t0, t1] * len(blocks)
    return ctx, tabs, ws


def _oracle_chain(oracle, cfg, blocks):
    p0 = oracle.partition(cfg["coords"], cfg["batch"], cfg["grid"], cfg["window"], cfg["set_size"], 0)
    p1 = oracle.partition(cfg["coords"], cfg["batch"], cfg["grid"], cfg["window"], cfg["set_size"], 1)
    x = cfg["feats"].astype(np.float64)
    for blk in blocks:
        x = oracle.block(x, p0.set_table, p1.set_table, blk)
    return x


@pytest.mark.parametrize("n,n_blocks", [(6000, 4), (300, 2), (40, 3)])
def test_chain_is_bitwise_the_layers_one_by_one_and_matches_the_oracle(gpu, oracle, n, n_blocks):
    """Eight (four, six) layers in one launch: every tile does the arithmetic it does in a launch of its own layer,
    so the chain's output is bitwise that of dsvt_layer called layer after layer; both match the oracle.  With 300
    or 40 voxels a layer has fewer tiles than the launch has thread blocks: most blocks' first tile belongs to a
    later layer and has to wait for the rows it reads."""
    cfg = di.make_config(2, n_override=n)
    blocks = cfg["blocks"][:n_blocks]
    ctx, tabs, ws = _setup(gpu, cfg, blocks)
    x = dev(cfg["feats"])
    y = torch.empty_like(x)
    ctx.layers(x, tabs, ws, y)
    assert ctx.status_sync() == 0
    z = torch.empty_like(x)
    src = x
    for t, w in zip(tabs, ws):
        ctx.layer(src, t, w, z)
        src = z
    assert ctx.status_sync() == 0
    assert torch.equal(y, z)
    check_close(y.cpu().numpy(), _oracle_chain(oracle, cfg, blocks), "bf16", "chain of %d layers" % len(ws))
    # in place, and again (the launch's counters and stamps are per launch)
    for _ in range(2):
        w_ = x.clone()
        ctx.layers(w_, tabs, ws, w_)
        assert ctx.status_sync() == 0
        assert torch.equal(w_, y)


def test_chain_without_a_tile_plan(gpu, oracle):
    """Row offsets whose plan entry says "no plan" (a caller that filled them by hand): tiles are cut by row
    ranges instead.  Same sets, other tiles: results agree with the oracle, and with the planned run closely."""
    cfg = di.make_config(2, n_override=5000)
    blocks = cfg["blocks"][:2]
    ctx, tabs, ws = _setup(gpu, cfg, blocks)
    x = dev(cfg["feats"])
    y = torch.empty_like(x)
    ctx.layers(x, tabs, ws, y)
    for t in tabs[:2]:
        t.set_rowoff[t.cap_sets + 1] = -1
    z = torch.empty_like(x)
    ctx.layers(x, tabs, ws, z)
    assert ctx.status_sync() == 0
    want = _oracle_chain(oracle, cfg, blocks)
    check_close(z.cpu().numpy(), want, "bf16", "chain without a plan")
    check_close(y.cpu().numpy(), want, "bf16", "chain with a plan")
    assert float((y - z).abs().max()) <= 2e-2 * float(np.abs(want).max())


@pytest.mark.parametrize("window,tau,n", [((1, 1, 1), 36, 1500), ((2, 1, 1), 36, 2500), ((8, 8, 1), 64, 4096)])
def test_chain_on_extreme_tile_plans(gpu, oracle, window, tau, n):
    """Tiles at the limits of the plan: every voxel a window (and a set) of its own, 128 one-row sets per tile;
    sets of one or two rows; and full windows whose 64-row sets fill a tile in pairs."""
    cfg = di.random_case(5, n, (64, 64, 1), window, tau, 192, 8, hidden=384, layernorm=True, bf16=True, n_blocks=2)
    ctx, tabs, ws = _setup(gpu, cfg, cfg["blocks"])
    x = dev(cfg["feats"])
    y = torch.empty_like(x)
    ctx.layers(x, tabs, ws, y)
    assert ctx.status_sync() == 0
    check_close(y.cpu().numpy(), _oracle_chain(oracle, cfg, cfg["blocks"]), "bf16", "chain, window %s" % (window,))


def test_chain_with_other_tables_per_block(gpu, oracle):
    """Hybrid windows: the second block runs on the tables of another window cut, so a tile of its first layer
    reads rows that tiles anywhere in the previous layer wrote (the stamps are per voxel, not per window)."""
    cfg = di.make_config(2, n_override=4000)
    blocks = cfg["blocks"][:2]
    ctx = gpu.Context(cfg["n"], 4 * _nwin(cfg), cfg["C"])
    dc = dev(cfg["coords"])
    a0, a1 = ctx.partition_rotated(dc, 1, cfg["grid"], (12, 12, 1), 36)
    b0, b1 = ctx.partition_rotated(dc, 1, cfg["grid"], (24, 24, 1), 36, shift=(12, 12, 0))
    ws = [gpu.device_weights(l, precision_of(cfg), ctx.device) for blk in blocks for l in blk]
    x = dev(cfg["feats"])
    y = torch.empty_like(x)
    ctx.layers(x, [a0, a1, b0, b1], ws, y)
    assert ctx.status_sync() == 0
    pa = [oracle.partition(cfg["coords"], 1, cfg["grid"], (12, 12, 1), 36, ax).set_table for ax in (0, 1)]
    pb = [oracle.partition(cfg["coords"], 1, cfg["grid"], (24, 24, 1), 36, ax, shift=(12, 12, 0)).set_table
          for ax in (0, 1)]
    want = oracle.block(oracle.block(cfg["feats"], pa[0], pa[1], blocks[0]), pb[0], pb[1], blocks[1])
    check_close(y.cpu().numpy(), want, "bf16", "two blocks on two window cuts")


def test_a_row_no_earlier_layer_wrote_ends_a_bounded_wait(gpu):
    """A later layer that reads a voxel the layer before it never wrote breaks the call's contract: the wait for
    that row's stamp is bounded and ends with DSVT_STATUS_TIMEOUT; the context stays usable.  (Dropping a set from
    the first layer's plan leaves its voxels unwritten.)"""
    cfg = di.make_config(2, n_override=600)
    ctx, tabs, ws = _setup(gpu, cfg, cfg["blocks"][:1])
    x = dev(cfg["feats"])
    y = torch.empty_like(x)
    ctx.layers(x, tabs, ws, y)
    assert ctx.status_sync() == 0
    # the first layer's table loses its last set: that set's voxels are never stamped
    short = gpu.SetTable(tabs[0].set_table, tabs[0].num_sets.clone(), tabs[0].set_rowoff.clone(), tabs[0].cap_sets,
                         tabs[0].set_size)
    S = int(short.num_sets.item())
    short.num_sets[0] = S - 1
    plan0 = short.cap_sets + 1
    nt = int(short.set_rowoff[plan0].item()) & ~0x40000000  # (the flag of a plan over reordered sets)
    short.set_rowoff[plan0 + 1 + nt] = S - 1  # the last tile ends one set earlier
    z = torch.empty_like(x)
    ctx.layers(x, [short, tabs[1]], ws, z)
    assert ctx.status_sync() & gpu.STATUS_TIMEOUT
    ctx.layers(x, tabs, ws, z)
    assert ctx.status_sync() == 0
    assert torch.equal(z, y)


def test_positional_term_on_the_tensor_core_path(gpu, oracle):
    """An additive positional term (added to the input of the query and key maps only, not to the values) with
    bfloat16 weights: one layer alone, attention alone, and a chain of four layers, each against the oracle."""
    cfg = di.make_config(2, n_override=5000)
    blocks = cfg["blocks"][:2]
    ctx, tabs, ws = _setup(gpu, cfg, blocks)
    rng = np.random.default_rng(11)
    pe = (0.5 * rng.standard_normal((cfg["n"], cfg["C"]))).astype(np.float32)
    x, dpe = dev(cfg["feats"]), dev(pe)
    p0 = oracle.partition(cfg["coords"], 1, cfg["grid"], cfg["window"], cfg["set_size"], 0).set_table
    p1 = oracle.partition(cfg["coords"], 1, cfg["grid"], cfg["window"], cfg["set_size"], 1).set_table
    y = torch.empty_like(x)
    ctx.layer(x, tabs[0], ws[0], y, pe=dpe)
    assert ctx.status_sync() == 0
    check_close(y.cpu().numpy(), oracle.layer(cfg["feats"], p0, blocks[0][0], pe=pe), "bf16", "layer with a term")
    ctx.set_attention(x, tabs[0], ws[0], y, pe=dpe)
    assert ctx.status_sync() == 0
    l0 = blocks[0][0]
    want, _ = oracle.set_attention(cfg["feats"], p0, l0["W_qkv"], l0["b_qkv"], l0["W_o"], l0["b_o"], l0["heads"], pe=pe)
    rows = np.unique(p0)
    check_close(y.cpu().numpy()[rows], want[rows], "bf16", "attention with a term")
    ctx.layers(x, tabs, ws, y, pe=dpe)
    assert ctx.status_sync() == 0
    w = cfg["feats"].astype(np.float64)
    for blk in blocks:
        w = oracle.block(w, p0, p1, blk, pe=pe)
    check_close(y.cpu().numpy(), w, "bf16", "chain with a term")
    # and the term matters: without it the result is another one
    z = torch.empty_like(x)
    ctx.layers(x, tabs, ws, z)
    assert float((y - z).abs().max()) > 1e-2
