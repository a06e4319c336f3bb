"""Pins for the oracle's attention-style 3D pooling (Eq. 6, Eq. 7). CPU only."""
import numpy as np
import pytest
import torch

import dsvt_inputs as di


def _softmax(a):
    e = np.exp(a - a.max())
    return e / e.sum()


def _brute_pool(coords, feats, grid, pool, Wt, heads, mask_empty, slot_pe=None):
    """Independent restatement with a python dict of regions."""
    l, w, h = pool
    C = feats.shape[1]
    d = C // heads
    regions = {}
    for i, (b, x, y, z) in enumerate(coords.tolist()):
        regions.setdefault((b, x // l, y // w, z // h), {})[((x % l) * w + y % w) * h + z % h] = i
    f64 = lambda k: np.asarray(Wt[k], dtype=np.float64)
    oc, of = [], []
    for key in sorted(regions):
        dense = np.zeros((l * w * h, C))
        occ = np.zeros(l * w * h, dtype=bool)
        for s, i in regions[key].items():
            dense[s] = feats[i]
            occ[s] = True
        use = occ if mask_empty else np.ones_like(occ)
        P = dense[use].max(axis=0)
        kv_in = dense if slot_pe is None else dense + slot_pe
        q = f64("W_q") @ P + f64("b_q")
        K = kv_in @ f64("W_k").T + f64("b_k")
        V = kv_in @ f64("W_v").T + f64("b_v")
        att = np.zeros(C)
        for hh in range(heads):
            sl = slice(hh * d, (hh + 1) * d)
            a = _softmax((K[use][:, sl] @ q[sl]) / np.sqrt(d))
            att[sl] = a @ V[use][:, sl]
        oc.append(key)
        of.append(f64("W_o") @ att + f64("b_o"))
    return np.array(oc, dtype=np.int32), np.array(of)


@pytest.mark.parametrize("mask_empty", [0, 1])
@pytest.mark.parametrize("grid,pool,batch,n,with_pe", [
    ((16, 16, 1), (2, 2, 1), 1, 120, False),
    ((9, 7, 8), (2, 2, 2), 2, 400, True),
    ((6, 6, 8), (1, 1, 4), 1, 150, False),
])
def test_pool_vs_brute_force(oracle, grid, pool, batch, n, with_pe, mask_empty):
    rng = np.random.default_rng(17)
    C, heads = 16, 4
    coords = di.unique_cells(rng, n, grid, batch)
    feats = rng.standard_normal((n, C))
    nslots = pool[0] * pool[1] * pool[2]
    Wt = di.make_pool_weights(rng, C, heads, False, nslots, with_pe)
    got = oracle.pool(coords, feats, batch, grid, pool, Wt["W_q"], Wt["W_k"], Wt["W_v"], Wt["W_o"],
                      Wt["b_q"], Wt["b_k"], Wt["b_v"], Wt["b_o"], heads, slot_pe=Wt["slot_pe"], mask_empty=mask_empty)
    pe = None if Wt["slot_pe"] is None else Wt["slot_pe"].astype(np.float64)
    wc, wf = _brute_pool(coords, feats, grid, pool, Wt, heads, mask_empty, pe)
    assert np.array_equal(got.coords, wc)
    assert np.abs(got.feats - wf).max() < 1e-12
    # region_of / slot_of are consistent with the output coords
    assert np.array_equal(got.coords[got.region_of][:, 1], coords[:, 1] // pool[0])
    assert np.array_equal(got.coords[got.region_of][:, 3], coords[:, 3] // pool[2])
    assert np.array_equal(got.slot_of, ((coords[:, 1] % pool[0]) * pool[1] + coords[:, 2] % pool[1]) * pool[2]
                          + coords[:, 3] % pool[2])
    # ascending region keys
    G = [-(-grid[a] // pool[a]) for a in range(3)]
    keys = ((got.coords[:, 0].astype(np.int64) * G[0] + got.coords[:, 1]) * G[1] + got.coords[:, 2]) * G[2] \
        + got.coords[:, 3]
    assert np.all(np.diff(keys) > 0)


def test_pool_max_is_torch_max_pool_over_padded_region(oracle):
    """Eq. 6 against torch's max_pool3d on the zero-padded dense grid (4x4x2, regions 2x2x2).
    With identity projections the output is softmax(<P, p_s>/sqrt(C)) . p_s, which depends on P."""
    rng = np.random.default_rng(2)
    C, heads = 4, 1
    grid, pool = (4, 4, 2), (2, 2, 2)
    coords = di.unique_cells(rng, 32, grid, 1)
    feats = rng.standard_normal((32, C))
    dense = np.zeros((4, 4, 2, C))
    dense[coords[:, 1], coords[:, 2], coords[:, 3]] = feats
    mp = torch.nn.functional.max_pool3d(torch.tensor(dense).permute(3, 0, 1, 2)[None], 2)[0].permute(1, 2, 3, 0)
    I = np.eye(C)
    z = np.zeros(C)
    got = oracle.pool(coords, feats, 1, grid, pool, I, I, I, I, z, z, z, z, heads)
    for r, (b, X, Y, Z) in enumerate(got.coords.tolist()):
        P = mp[X, Y, Z].numpy()
        slots = dense[2 * X:2 * X + 2, 2 * Y:2 * Y + 2, 2 * Z:2 * Z + 2].reshape(8, C)
        a = _softmax(slots @ P / np.sqrt(C))
        assert np.abs(got.feats[r] - a @ slots).max() < 1e-12


def test_pool_closed_forms(oracle):
    rng = np.random.default_rng(4)
    C, heads = 16, 4
    Wt = di.make_pool_weights(rng, C, heads, False)
    f64 = lambda k: np.asarray(Wt[k], dtype=np.float64)
    # (a) all four slots hold the same vector p: P = p, attention returns v(p): out = W_o (W_v p + b_v) + b_o
    p = rng.standard_normal(C)
    coords = np.array([[0, 2, 4, 0], [0, 3, 4, 0], [0, 2, 5, 0], [0, 3, 5, 0]], dtype=np.int32)
    feats = np.tile(p, (4, 1))
    got = oracle.pool(coords, feats, 1, (8, 8, 1), (2, 2, 1), Wt["W_q"], Wt["W_k"], Wt["W_v"], Wt["W_o"],
                      Wt["b_q"], Wt["b_k"], Wt["b_v"], Wt["b_o"], heads)
    want = f64("W_o") @ (f64("W_v") @ p + f64("b_v")) + f64("b_o")
    assert got.coords.tolist() == [[0, 1, 2, 0]]
    assert np.abs(got.feats[0] - want).max() < 1e-13
    # (b) W_q = 0, b_q = 0: uniform weights over the slots that take part
    feats = rng.standard_normal((3, C))
    coords = np.array([[0, 0, 0, 0], [0, 1, 1, 0], [0, 0, 1, 0]], dtype=np.int32)  # slot (1,0) is empty
    Z, zb = np.zeros((C, C)), np.zeros(C)
    vals = feats @ f64("W_v").T + f64("b_v")
    dense_mean = (vals.sum(axis=0) + f64("b_v")) / 4.0  # the empty slot contributes v(0) = b_v
    for mask_empty, mean in ((0, dense_mean), (1, vals.mean(axis=0))):
        got = oracle.pool(coords, feats, 1, (8, 8, 1), (2, 2, 1), Z, Wt["W_k"], Wt["W_v"], Wt["W_o"],
                          zb, Wt["b_k"], Wt["b_v"], Wt["b_o"], heads, mask_empty=mask_empty)
        assert np.abs(got.feats[0] - (f64("W_o") @ mean + f64("b_o"))).max() < 1e-13


def test_pool_padded_max_includes_zero_rows(oracle):
    """Default mode pads the region to dense before the max (text of Eq. 6): with one all-negative
    voxel in a 2x2x1 region P = 0, so q = b_q; the masked mode gives P = the voxel itself."""
    C, heads = 8, 2
    rng = np.random.default_rng(6)
    Wt = di.make_pool_weights(rng, C, heads, False)
    f64 = lambda k: np.asarray(Wt[k], dtype=np.float64)
    x = -np.abs(rng.standard_normal((1, C))) - 0.5
    coords = np.array([[0, 1, 0, 0]], dtype=np.int32)
    args = (Wt["W_q"], Wt["W_k"], Wt["W_v"], Wt["W_o"], Wt["b_q"], Wt["b_k"], Wt["b_v"], Wt["b_o"], heads)
    masked = oracle.pool(coords, x, 1, (2, 2, 1), (2, 2, 1), *args, mask_empty=1)
    assert np.abs(masked.feats[0] - (f64("W_o") @ (f64("W_v") @ x[0] + f64("b_v")) + f64("b_o"))).max() < 1e-13
    dense = oracle.pool(coords, x, 1, (2, 2, 1), (2, 2, 1), *args, mask_empty=0)
    d = C // heads
    q = f64("b_q")  # W_q * 0 + b_q
    slots = np.zeros((4, C)); slots[2] = x[0]  # slot = (x%2)*2 + y%2 = 2
    K = slots @ f64("W_k").T + f64("b_k")
    V = slots @ f64("W_v").T + f64("b_v")
    att = np.concatenate([_softmax(K[:, h * d:(h + 1) * d] @ q[h * d:(h + 1) * d] / np.sqrt(d)) @ V[:, h * d:(h + 1) * d]
                          for h in range(heads)])
    assert np.abs(dense.feats[0] - (f64("W_o") @ att + f64("b_o"))).max() < 1e-13


def test_pool_errors(oracle):
    C = 4
    I, z = np.eye(C), np.zeros(C)
    dup = np.array([[0, 1, 1, 0], [0, 1, 1, 0]], dtype=np.int32)
    with pytest.raises(ValueError):
        oracle.pool(dup, np.zeros((2, C)), 1, (4, 4, 1), (2, 2, 1), I, I, I, I, z, z, z, z, 1)
    out = np.array([[0, 4, 1, 0]], dtype=np.int32)
    with pytest.raises(ValueError):
        oracle.pool(out, np.zeros((1, C)), 1, (4, 4, 1), (2, 2, 1), I, I, I, I, z, z, z, z, 1)
