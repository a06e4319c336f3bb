"""Seeded generators for the five workload configurations and for small test cases.

The paper measures on Waymo Open frames (0.32 m pillars over +-74.88 m, i.e. a
468 x 468 grid; windows 12 x 12, set size 36, 192 channels, 8 heads, 384 hidden
channels, four blocks: Sec. 4.1 and Appendix B.1.1).  That dataset is not
available here; the generators below produce synthetic LiDAR-shaped voxel sets
with those shapes and stand in for it.

Every generator is a pure function of its seed (numpy PCG64).
"""
from __future__ import annotations

import math
from typing import Dict, List, Optional

import numpy as np

CONFIG_IDS = (1, 2, 3, 4, 5)

CELL = 0.32  # metres per cell
HALF_RANGE = 74.88  # metres; 2 * 74.88 / 0.32 = 468 cells


# ---------------------------------------------------------------------------
# dtype helpers (storage formats only)
# ---------------------------------------------------------------------------
def round_bf16(a: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even); returns float32."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    r = ((u >> 16) & 1) + 0x7FFF
    u2 = ((u + r) & 0xFFFF0000).astype(np.uint32)
    return u2.view(np.float32).reshape(np.shape(a))


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """uint16 storage of float32 values that are already bfloat16-representable."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    assert not np.any(u & 0xFFFF), "values are not bfloat16-representable"
    return (u >> 16).astype(np.uint16).reshape(np.shape(a))


# ---------------------------------------------------------------------------
# weights
# ---------------------------------------------------------------------------
def _xavier(rng, out_f: int, in_f: int) -> np.ndarray:
    a = math.sqrt(6.0 / (in_f + out_f))
    return rng.uniform(-a, a, size=(out_f, in_f)).astype(np.float32)


def _bias(rng, k: int) -> np.ndarray:
    return rng.uniform(-0.02, 0.02, size=(k,)).astype(np.float32)


def make_layer(rng, C: int, heads: int, hidden: int, layernorm: bool, bf16: bool) -> Dict:
    """One DSVT layer's parameters.  hidden == 0: no MLP; layernorm False: no LN."""
    cast = round_bf16 if bf16 else (lambda a: a)
    p: Dict = {"C": C, "heads": heads, "hidden": hidden, "ln_eps": 1e-5}
    # Q, K, V are separate C x C maps stacked into one [3C][C] matrix
    p["W_qkv"] = cast(np.concatenate([_xavier(rng, C, C) for _ in range(3)], axis=0))
    p["b_qkv"] = _bias(rng, 3 * C)
    p["W_o"] = cast(_xavier(rng, C, C))
    p["b_o"] = _bias(rng, C)
    if hidden > 0:
        p["W_1"] = cast(_xavier(rng, hidden, C))
        p["b_1"] = _bias(rng, hidden)
        p["W_2"] = cast(_xavier(rng, C, hidden))
        p["b_2"] = _bias(rng, C)
    else:
        p["W_1"] = p["b_1"] = p["W_2"] = p["b_2"] = None
    if layernorm:
        for k in ("ln1", "ln2"):
            p[k + "_g"] = (1.0 + 0.1 * rng.standard_normal(C)).astype(np.float32)
            p[k + "_b"] = (0.1 * rng.standard_normal(C)).astype(np.float32)
    else:
        p["ln1_g"] = p["ln1_b"] = p["ln2_g"] = p["ln2_b"] = None
    return p


def make_pool_weights(rng, C: int, heads: int, bf16: bool, nslots: int = 0, slot_pe: bool = False) -> Dict:
    cast = round_bf16 if bf16 else (lambda a: a)
    p: Dict = {"C": C, "heads": heads}
    for k in ("q", "k", "v", "o"):
        p["W_" + k] = cast(_xavier(rng, C, C))
        p["b_" + k] = _bias(rng, C)
    p["slot_pe"] = (0.1 * rng.standard_normal((nslots, C))).astype(np.float32) if slot_pe else None
    return p


# ---------------------------------------------------------------------------
# coordinates
# ---------------------------------------------------------------------------
def unique_cells(rng, n: int, grid, batch: int = 1) -> np.ndarray:
    """n distinct cells drawn uniformly without replacement; int32 [n][4] = (b,x,y,z) in draw order."""
    gx, gy, gz = (int(g) for g in grid)
    total = batch * gx * gy * gz
    assert 0 <= n <= total
    flat = rng.permutation(total)[:n].astype(np.int64)
    z = flat % gz
    y = (flat // gz) % gy
    x = (flat // (gz * gy)) % gx
    b = flat // (gz * gy * gx)
    return np.stack([b, x, y, z], axis=1).astype(np.int32)


def _lidar_points(rng, k: int):
    """k points (x, y in metres) and a flag saying which are ring points.

    Half are 'ring' points: ring j of 64 has radius 3 * 25**(j/63) m plus
    N(0, 0.1 m) jitter and a uniform azimuth.  Half are 'clutter' with areal
    density proportional to 1/r^2, i.e. log-uniform radius on [2, 105.9] m.
    """
    is_ring = rng.random(k) < 0.5
    ring = rng.integers(0, 64, size=k)
    r_ring = 3.0 * np.power(25.0, ring / 63.0) + 0.1 * rng.standard_normal(k)
    r_clut = np.exp(rng.uniform(math.log(2.0), math.log(105.9), size=k))
    r = np.where(is_ring, r_ring, r_clut)
    az = rng.uniform(0.0, 2.0 * math.pi, size=k)
    return r * np.cos(az), r * np.sin(az), is_ring


def _first_unique(keys: np.ndarray, limit: int) -> np.ndarray:
    """Indices (ascending, i.e. draw order) of the first occurrence of each key, at most `limit`."""
    _, first = np.unique(keys, return_index=True)
    first.sort()
    return first[:limit]


def lidar_pillars(rng, n: int, grid_xy: int = 468, half_range: float = HALF_RANGE, cell: float = CELL) -> np.ndarray:
    """Exactly n distinct (x, y) cells of a LiDAR-shaped frame, in draw order.  int64 [n][2]."""
    cells = np.zeros((0, 2), dtype=np.int64)
    while True:
        px, py, _ = _lidar_points(rng, 2 * n)
        ok = (np.abs(px) < half_range) & (np.abs(py) < half_range)
        cx = np.floor((px[ok] + half_range) / cell).astype(np.int64)
        cy = np.floor((py[ok] + half_range) / cell).astype(np.int64)
        ok2 = (cx >= 0) & (cx < grid_xy) & (cy >= 0) & (cy < grid_xy)
        cells = np.concatenate([cells, np.stack([cx[ok2], cy[ok2]], axis=1)], axis=0)
        keep = _first_unique(cells[:, 0] * grid_xy + cells[:, 1], n)
        cells = cells[keep]
        if cells.shape[0] >= n:
            return cells[:n]


def lidar_voxels(rng, n: int, grid_xy: int = 468, grid_z: int = 32) -> np.ndarray:
    """Exactly n distinct (x, y, z) voxels: ring points sit in slices {0, 1}; each clutter point
    is a column from slice 0 upward of height 1 + Geometric(1/2), capped at 8."""
    vox = np.zeros((0, 3), dtype=np.int64)
    while True:
        k = n
        px, py, is_ring = _lidar_points(rng, k)
        zr = rng.integers(0, 2, size=k)
        height = np.minimum(rng.geometric(0.5, size=k), 8)  # 1 + Geometric(1/2) counted from 0, capped at 8
        ok = (np.abs(px) < HALF_RANGE) & (np.abs(py) < HALF_RANGE)
        cx = np.floor((px + HALF_RANGE) / CELL).astype(np.int64)
        cy = np.floor((py + HALF_RANGE) / CELL).astype(np.int64)
        ok &= (cx >= 0) & (cx < grid_xy) & (cy >= 0) & (cy < grid_xy)
        rows: List[np.ndarray] = []
        # emit voxels point by point, keeping draw order: ring -> one voxel, clutter -> a column
        reps = np.where(is_ring, 1, height)
        reps = np.where(ok, reps, 0)
        idx = np.repeat(np.arange(k), reps)
        first = np.cumsum(reps) - reps
        level = np.arange(idx.shape[0]) - np.repeat(first, reps)
        z = np.where(is_ring[idx], zr[idx], level)
        rows.append(np.stack([cx[idx], cy[idx], z], axis=1))
        vox = np.concatenate([vox] + rows, axis=0)
        keys = (vox[:, 0] * grid_xy + vox[:, 1]) * grid_z + vox[:, 2]
        vox = vox[_first_unique(keys, n)]
        if vox.shape[0] >= n:
            return vox[:n]


def skewed_pillars(rng, n: int = 200_000, grid_xy: int = 936, win: int = 12) -> np.ndarray:
    """Occupancy-skewed frame: 5 % of the windows are full (win*win voxels), 60 % hold 1..3,
    the rest share the remainder (each 4..win*win-1).  Returns int64 [n][2] cells."""
    nw_side = grid_xy // win
    nw = nw_side * nw_side
    vol = win * win
    n_full = int(round(0.05 * nw))
    n_tiny = int(round(0.60 * nw))
    n_mid = nw - n_full - n_tiny
    roles = rng.permutation(nw)
    counts = np.zeros(nw, dtype=np.int64)
    counts[roles[:n_full]] = vol
    counts[roles[n_full:n_full + n_tiny]] = rng.integers(1, 4, size=n_tiny)
    rem = n - int(counts.sum())
    mid = rng.integers(4, vol, size=n_mid)  # 4 .. vol-1
    diff = rem - int(mid.sum())
    assert 4 * n_mid <= rem <= (vol - 1) * n_mid, "remainder does not fit the middle windows"
    while diff != 0:
        step = 1 if diff > 0 else -1
        room = np.flatnonzero((mid + step >= 4) & (mid + step <= vol - 1))
        pick = rng.permutation(room)[: min(abs(diff), room.shape[0])]
        mid[pick] += step
        diff -= step * pick.shape[0]
    counts[roles[n_full + n_tiny:]] = mid
    assert int(counts.sum()) == n
    # cells inside each window: uniform without replacement (argsort of random keys)
    out = np.zeros((n, 2), dtype=np.int64)
    pos = 0
    scores = rng.random((nw, vol))
    order = np.argsort(scores, axis=1)
    for w in range(nw):
        c = int(counts[w])
        if c == 0:
            continue
        cells = order[w, :c]
        wx, wy = divmod(w, nw_side)
        out[pos:pos + c, 0] = wx * win + cells // win
        out[pos:pos + c, 1] = wy * win + cells % win
        pos += c
    # voxel order in memory is arbitrary: shuffle so that nothing downstream relies on window order
    return out[rng.permutation(n)]


def _coords4(b, xy_or_xyz: np.ndarray) -> np.ndarray:
    n = xy_or_xyz.shape[0]
    out = np.zeros((n, 4), dtype=np.int32)
    out[:, 0] = b
    out[:, 1] = xy_or_xyz[:, 0]
    out[:, 2] = xy_or_xyz[:, 1]
    if xy_or_xyz.shape[1] > 2:
        out[:, 3] = xy_or_xyz[:, 2]
    return out


# ---------------------------------------------------------------------------
# the five configurations
# ---------------------------------------------------------------------------
def make_config(cid: int, n_override: Optional[int] = None, with_feats: bool = True) -> Dict:
    """Configuration `cid` (1..5; 6 = the nuScenes-shaped extra; 7 = the DSVT-V stage layout: `stages`, `pools`) as a dict.

    Keys: id, name, batch, grid, window, set_size, C, heads, hidden, precision
    ('fp32' | 'bf16'), coords int32 [n][4], feats float32 [n][C], blocks (list of
    [layer_x, layer_y] parameter dicts) and, for config 5, pool / pool_shape /
    blocks_after_pool.  n_override scales the voxel count (same recipe) for tests.
    """
    seed = 1000 + cid
    rng = np.random.default_rng(seed)
    cfg: Dict = {"id": cid, "seed": seed}
    if cid == 1:
        n = n_override or 2000
        cfg.update(name="tiny", batch=1, grid=(64, 64, 1), window=(12, 12, 1), set_size=36, C=128, heads=8,
                   hidden=0, layernorm=False, precision="fp32", n_blocks=1)
        cfg["coords"] = unique_cells(rng, n, cfg["grid"], 1)
    elif cid == 2:
        n = n_override or 32_000
        cfg.update(name="waymo_pillars", batch=1, grid=(468, 468, 1), window=(12, 12, 1), set_size=36, C=192,
                   heads=8, hidden=384, layernorm=True, precision="bf16", n_blocks=4)
        cfg["coords"] = _coords4(0, lidar_pillars(rng, n))
    elif cid == 3:
        n = n_override or 120_000
        cfg.update(name="voxels_3d", batch=1, grid=(468, 468, 32), window=(12, 12, 32), set_size=36, C=192,
                   heads=8, hidden=384, layernorm=True, precision="bf16", n_blocks=4)
        cfg["coords"] = _coords4(0, lidar_voxels(rng, n))
    elif cid == 4:
        per = (n_override or 128_000) // 4
        cfg.update(name="batched_pillars", batch=4, grid=(468, 468, 1), window=(12, 12, 1), set_size=36, C=192,
                   heads=8, hidden=384, layernorm=True, precision="bf16", n_blocks=4)
        frames = []
        for b in range(4):
            frng = np.random.default_rng(seed + b)
            frames.append(_coords4(b, lidar_pillars(frng, per)))
        cfg["coords"] = np.concatenate(frames, axis=0)
    elif cid == 5:
        n = n_override or 200_000
        cfg.update(name="skew_pool", batch=1, grid=(936, 936, 1), window=(12, 12, 1), set_size=36, C=192,
                   heads=8, hidden=384, layernorm=True, precision="bf16", n_blocks=2,
                   pool_shape=(2, 2, 1), n_blocks_after_pool=2)
        cfg["coords"] = _coords4(0, skewed_pillars(rng, n))
    elif cid == 6:
        # the paper's second workload shape (Appendix B.1.2: windows 30 x 30 x 1, set size 90, 128 channels, 8 heads,
        # 256 hidden channels).  The paper does not state the pillar size there: 0.3 m cells over +-54 m (360 x 360)
        # and 30 000 pillars are this generator's choice.  Not one of the five measured configurations.
        n = n_override or 30_000
        cfg.update(name="nuscenes_pillars", batch=1, grid=(360, 360, 1), window=(30, 30, 1), set_size=90, C=128,
                   heads=8, hidden=256, layernorm=True, precision="bf16", n_blocks=4)
        cfg["coords"] = _coords4(0, lidar_pillars(rng, n, 360, 54.0, 0.3))
    elif cid == 7:
        # the voxel variant's stage layout (Appendix B.1.1, DSVT-V): four stages of one block each, windows of
        # 32 / 8 / 2 / 1 cells along z (12 x 12 in x, y), attention-style pooling along z with strides 4, 4, 2
        # between them, set size 48.  Same voxel generator as configuration 3.  Not one of the five measured
        # configurations.
        n = n_override or 120_000
        cfg.update(name="dsvt_v_stages", batch=1, grid=(468, 468, 32), window=(12, 12, 32), set_size=48, C=192,
                   heads=8, hidden=384, layernorm=True, precision="bf16", n_blocks=1)
        cfg["coords"] = _coords4(0, lidar_voxels(rng, n))
    else:
        raise ValueError("config id must be 1..7")
    n = cfg["coords"].shape[0]
    cfg["n"] = n
    C = cfg["C"]
    bf16 = cfg["precision"] == "bf16"
    wrng = np.random.default_rng(seed * 7919 + 1)
    cfg["feats"] = wrng.standard_normal((n, C), dtype=np.float32) if with_feats else None
    cfg["blocks"] = [
        [make_layer(wrng, C, cfg["heads"], cfg["hidden"], cfg["layernorm"], bf16) for _ in range(2)]
        for _ in range(cfg["n_blocks"])
    ]
    if cid == 7:
        z_windows, strides = (32, 8, 2, 1), (4, 4, 2)
        cfg["stages"] = [{"window": (12, 12, z_windows[0]), "blocks": cfg["blocks"]}]
        cfg["pools"] = []
        for i, st in enumerate(strides):
            cfg["pools"].append({"shape": (1, 1, st), "weights": make_pool_weights(wrng, C, cfg["heads"], bf16)})
            cfg["stages"].append({"window": (12, 12, z_windows[i + 1]),
                                  "blocks": [[make_layer(wrng, C, cfg["heads"], cfg["hidden"], True, bf16)
                                              for _ in range(2)]]})
    if cid == 5:
        cfg["pool"] = make_pool_weights(wrng, C, cfg["heads"], bf16)
        cfg["blocks_after_pool"] = [
            [make_layer(wrng, C, cfg["heads"], cfg["hidden"], True, bf16) for _ in range(2)]
            for _ in range(cfg["n_blocks_after_pool"])
        ]
    return cfg


def random_case(seed: int, n: int, grid, window, set_size: int, C: int, heads: int, hidden: int = 0,
                layernorm: bool = False, bf16: bool = False, batch: int = 1, n_blocks: int = 1) -> Dict:
    """A small uniform-random case with the same dict layout as make_config."""
    rng = np.random.default_rng(seed)
    cfg: Dict = dict(id=0, name="random", seed=seed, batch=batch, grid=tuple(grid), window=tuple(window),
                     set_size=set_size, C=C, heads=heads, hidden=hidden, layernorm=layernorm,
                     precision="bf16" if bf16 else "fp32", n_blocks=n_blocks, n=n)
    cfg["coords"] = unique_cells(rng, n, grid, batch)
    cfg["feats"] = rng.standard_normal((n, C), dtype=np.float32)
    cfg["blocks"] = [[make_layer(rng, C, heads, hidden, layernorm, bf16) for _ in range(2)] for _ in range(n_blocks)]
    return cfg
