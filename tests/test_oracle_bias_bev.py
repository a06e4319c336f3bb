"""Pins for the oracle's relative position bias (the Swin mechanism the text after Eq. 5 points to) and for the BEV
projection (Sec. 3.1).  CPU only."""
import os

import numpy as np
import pytest

import dsvt_inputs as di

GOLD = os.path.join(os.path.dirname(__file__), "golden")
NEG = -1.0e4  # a logit this far below the others has softmax weight exp(-1e4) == 0 in double precision


def _case(seed, n, grid, window, tau, C, heads):
    cfg = di.random_case(seed, n, grid, window, tau, C, heads)
    L = dict(cfg["blocks"][0][0])
    return cfg, cfg["feats"].astype(np.float64), L


def _attend(oracle, cfg, x, L, table, rpb, heads):
    out, covered = oracle.set_attention(x, table, L["W_qkv"], L["b_qkv"], L["W_o"], L["b_o"], heads, rpb=rpb,
                                        coords=cfg["coords"], rpb_extent=cfg["window"])
    assert covered.all()
    return out


def _value_path(x, L):
    """W_o (W_v x + b_v) + b_o for every voxel: what a query returns when it attends to exactly one key."""
    C = x.shape[1]
    Wv = np.asarray(L["W_qkv"], dtype=np.float64)[2 * C:]
    bv = np.asarray(L["b_qkv"], dtype=np.float64)[2 * C:]
    V = x @ Wv.T + bv
    return V, V @ np.asarray(L["W_o"], dtype=np.float64).T + np.asarray(L["b_o"], dtype=np.float64)


CASES = [(21, 110, (12, 12, 1), (6, 6, 1), 9, 16, 4), (22, 220, (8, 8, 4), (4, 4, 4), 12, 24, 2)]


@pytest.mark.parametrize("seed,n,grid,window,tau,C,heads", CASES)
def test_zero_and_constant_tables_change_nothing(oracle, seed, n, grid, window, tau, C, heads):
    cfg, x, L = _case(seed, n, grid, window, tau, C, heads)
    T = oracle.rel_bias_len(window)
    for axis in (0, 1):
        tab = oracle.partition(cfg["coords"], 1, grid, window, tau, axis).set_table
        plain, _ = oracle.set_attention(x, tab, L["W_qkv"], L["b_qkv"], L["W_o"], L["b_o"], heads)
        zero = _attend(oracle, cfg, x, L, tab, np.zeros((heads, T)), heads)
        assert np.array_equal(zero, plain)
        # softmax is invariant to a per-(head, query) shift of its logits
        const = _attend(oracle, cfg, x, L, tab, np.arange(1, heads + 1, dtype=np.float64)[:, None] * np.ones((1, T)), heads)
        assert np.abs(const - plain).max() < 1e-12


@pytest.mark.parametrize("seed,n,grid,window,tau,C,heads", CASES)
def test_table_that_admits_only_offset_zero_makes_every_voxel_attend_to_itself(oracle, seed, n, grid, window, tau, C, heads):
    cfg, x, L = _case(seed, n, grid, window, tau, C, heads)
    Lw, Ww, Hw = window
    B = np.full((heads, 2 * Lw - 1, 2 * Ww - 1, 2 * Hw - 1), NEG)
    B[:, Lw - 1, Ww - 1, Hw - 1] = 0.0
    tab = oracle.partition(cfg["coords"], 1, grid, window, tau, 0).set_table
    got = _attend(oracle, cfg, x, L, tab, B.reshape(heads, -1), heads)
    _, want = _value_path(x, L)
    assert np.abs(got - want).max() < 1e-12


@pytest.mark.parametrize("seed,n,grid,window,tau,C,heads", CASES)
@pytest.mark.parametrize("comp", [0, 1, 2])
def test_offset_is_query_minus_key_and_components_are_not_swapped(oracle, seed, n, grid, window, tau, C, heads, comp, sign=+1):
    """Only the offset +1 along one component is admitted: a query then returns the value of the member one cell
    below it along that component (coords[query] - coords[key] = +1), if its set holds one."""
    if window[comp] == 1:
        pytest.skip("no offset along a component of extent 1")
    cfg, x, L = _case(seed, n, grid, window, tau, C, heads)
    Lw, Ww, Hw = window
    B = np.full((heads, 2 * Lw - 1, 2 * Ww - 1, 2 * Hw - 1), NEG)
    centre = [Lw - 1, Ww - 1, Hw - 1]
    centre[comp] += 1
    B[:, centre[0], centre[1], centre[2]] = 0.0
    coords = cfg["coords"]
    _, vp = _value_path(x, L)
    checked = 0
    for axis in (0, 1):
        tab = oracle.partition(coords, 1, grid, window, tau, axis).set_table
        got = _attend(oracle, cfg, x, L, tab, B.reshape(heads, -1), heads)
        for row in tab:
            members = list(dict.fromkeys(row.tolist()))
            where = {tuple(coords[v, 1:]): v for v in members}
            for v in members:
                below = list(coords[v, 1:])
                below[comp] -= 1
                k = where.get(tuple(below))
                if k is not None:
                    assert np.abs(got[v] - vp[k]).max() < 1e-12
                    checked += 1
    assert checked > 10


def test_heads_read_their_own_table_rows(oracle):
    seed, n, grid, window, tau, C, heads = 23, 120, (12, 12, 1), (6, 6, 1), 12, 16, 2
    cfg, x, L = _case(seed, n, grid, window, tau, C, heads)
    L["W_o"] = np.eye(C)
    L["b_o"] = np.zeros(C)
    d = C // heads
    Lw, Ww, Hw = window
    B = np.full((heads, 2 * Lw - 1, 2 * Ww - 1, 2 * Hw - 1), NEG)
    B[0, Lw - 1, Ww - 1, Hw - 1] = 0.0  # head 0: itself
    B[1, Lw - 1, Ww, Hw - 1] = 0.0      # head 1: the member one cell below along y
    coords = cfg["coords"]
    V, _ = _value_path(x, L)
    tab = oracle.partition(coords, 1, grid, window, tau, 1).set_table
    got = _attend(oracle, cfg, x, L, tab, B.reshape(heads, -1), heads)
    assert np.abs(got[:, :d] - V[:, :d]).max() < 1e-12
    checked = 0
    for row in tab:
        members = list(dict.fromkeys(row.tolist()))
        where = {tuple(coords[v, 1:]): v for v in members}
        for v in members:
            k = where.get((coords[v, 1], coords[v, 2] - 1, coords[v, 3]))
            if k is not None:
                assert np.abs(got[v, d:] - V[k, d:]).max() < 1e-12
                checked += 1
    assert checked > 10


@pytest.mark.parametrize("seed,n,grid,window,tau,C,heads", CASES)
def test_random_table_against_dense_attention_with_a_bias_tensor(oracle, seed, n, grid, window, tau, C, heads):
    cfg, x, L = _case(seed, n, grid, window, tau, C, heads)
    rng = np.random.default_rng(seed + 100)
    Lw, Ww, Hw = window
    B = rng.standard_normal((heads, 2 * Lw - 1, 2 * Ww - 1, 2 * Hw - 1))
    coords = cfg["coords"].astype(np.int64)
    d = C // heads
    Wq, Wk, Wv = (np.asarray(L["W_qkv"], dtype=np.float64)[i * C:(i + 1) * C] for i in range(3))
    b = np.asarray(L["b_qkv"], dtype=np.float64)
    for axis in (0, 1):
        tab = oracle.partition(cfg["coords"], 1, grid, window, tau, axis).set_table
        got = _attend(oracle, cfg, x, L, tab, B.reshape(heads, -1), heads)
        want = np.zeros_like(got)
        for row in tab:
            m = list(dict.fromkeys(row.tolist()))
            X = x[m]
            Q, K, V = X @ Wq.T + b[:C], X @ Wk.T + b[C:2 * C], X @ Wv.T + b[2 * C:]
            off = coords[m][:, None, 1:] - coords[m][None, :, 1:] + np.array([Lw - 1, Ww - 1, Hw - 1])
            Y = np.zeros_like(Q)
            for h in range(heads):
                sl = slice(h * d, (h + 1) * d)
                A = Q[:, sl] @ K[:, sl].T / np.sqrt(d) + B[h][off[..., 0], off[..., 1], off[..., 2]]
                A = np.exp(A - A.max(axis=1, keepdims=True))
                Y[:, sl] = (A / A.sum(axis=1, keepdims=True)) @ V[:, sl]
            want[m] = Y @ np.asarray(L["W_o"], dtype=np.float64).T + np.asarray(L["b_o"], dtype=np.float64)
        assert np.abs(got - want).max() < 1e-12


def test_table_too_small_for_the_sets_is_refused(oracle):
    cfg, x, L = _case(24, 100, (12, 12, 1), (6, 6, 1), 9, 16, 4)
    tab = oracle.partition(cfg["coords"], 1, (12, 12, 1), (6, 6, 1), 9, 0).set_table
    with pytest.raises(ValueError):
        oracle.set_attention(x, tab, L["W_qkv"], L["b_qkv"], L["W_o"], L["b_o"], 4, rpb=np.zeros((4, 9)),
                             coords=cfg["coords"], rpb_extent=(2, 2, 1))


def test_layer_passes_the_bias_to_its_attention(oracle):
    seed, n, grid, window, tau, C, heads = 25, 110, (12, 12, 1), (6, 6, 1), 9, 16, 4
    cfg = di.random_case(seed, n, grid, window, tau, C, heads, hidden=32, layernorm=True)
    x = cfg["feats"].astype(np.float64)
    L = dict(cfg["blocks"][0][0])
    rng = np.random.default_rng(7)
    L["rpb"] = rng.standard_normal((heads, oracle.rel_bias_len(window)))
    L["rpb_extent"] = window
    tab = oracle.partition(cfg["coords"], 1, grid, window, tau, 0).set_table
    got = oracle.layer(x, tab, L, coords=cfg["coords"])
    z, _ = oracle.set_attention(x, tab, L["W_qkv"], L["b_qkv"], L["W_o"], L["b_o"], heads, rpb=L["rpb"],
                                coords=cfg["coords"], rpb_extent=window)

    def ln(v, g, bb):
        mu = v.mean(axis=1, keepdims=True)
        var = ((v - mu) ** 2).mean(axis=1, keepdims=True)
        return (v - mu) / np.sqrt(var + L.get("ln_eps", 1e-5)) * g + bb

    from scipy.special import erf
    x1 = ln(x + z, np.asarray(L["ln1_g"], dtype=np.float64), np.asarray(L["ln1_b"], dtype=np.float64))
    hmid = x1 @ np.asarray(L["W_1"], dtype=np.float64).T + np.asarray(L["b_1"], dtype=np.float64)
    hmid = 0.5 * hmid * (1.0 + erf(hmid / np.sqrt(2.0)))
    m = hmid @ np.asarray(L["W_2"], dtype=np.float64).T + np.asarray(L["b_2"], dtype=np.float64)
    want = ln(x1 + m, np.asarray(L["ln2_g"], dtype=np.float64), np.asarray(L["ln2_b"], dtype=np.float64))
    assert np.abs(got - want).max() < 1e-11
    plain = dict(L)
    plain.pop("rpb")
    assert np.abs(oracle.layer(x, tab, plain) - got).max() > 1e-3  # the bias is not silently dropped


# ---------------------------------------------------------------- BEV projection
def _read_bev():
    sec, data = None, {"coords": [], "feats": [], "map": []}
    for line in open(os.path.join(GOLD, "tiny_bev.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line in data:
            sec = line
            continue
        data[sec].append([float(t) for t in line.split()])
    return (np.array(data["coords"], dtype=np.int32), np.array(data["feats"]), np.array(data["map"]).reshape(1, 4, 2, 3))


def test_bev_hand_worked_example(oracle):
    coords, feats, want = _read_bev()
    got = oracle.bev_scatter(coords, feats, 1, (3, 2, 2))
    assert got.shape == (1, 4, 2, 3)
    assert np.array_equal(got, want)
    last = oracle.bev_scatter(coords, feats, 1, (3, 2, 2), channels_last=True)
    assert np.array_equal(last, want.transpose(0, 2, 3, 1))


@pytest.mark.parametrize("grid,batch,C", [((9, 7, 1), 2, 5), ((6, 5, 3), 3, 4)])
def test_bev_equals_indexed_assignment(oracle, grid, batch, C):
    rng = np.random.default_rng(5)
    n = 70
    coords = di.unique_cells(rng, n, grid, batch)
    feats = rng.standard_normal((n, C))
    X, Y, Z = grid
    got = oracle.bev_scatter(coords, feats, batch, grid)
    vol = np.zeros((batch, C, Z, Y, X))
    vol[coords[:, 0], :, coords[:, 3], coords[:, 2], coords[:, 1]] = feats
    assert np.array_equal(got, vol.reshape(batch, C * Z, Y, X))
    assert np.count_nonzero(got) == np.count_nonzero(feats)
    assert np.array_equal(oracle.bev_scatter(coords, feats, batch, grid, channels_last=True), got.transpose(0, 2, 3, 1))


def test_bev_refuses_two_voxels_in_one_cell(oracle):
    coords = np.array([[0, 1, 1, 0], [0, 1, 1, 0]], dtype=np.int32)
    with pytest.raises(ValueError):
        oracle.bev_scatter(coords, np.ones((2, 3)), 1, (4, 4, 1))
