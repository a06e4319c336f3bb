"""Pins for the oracle's set attention, layer and block (Eq. 4, Eq. 5, Appendix B.1.1). CPU only."""
import numpy as np
import pytest
import torch

import dsvt_inputs as di


def _softmax(a, axis=-1):
    a = a - a.max(axis=axis, keepdims=True)
    e = np.exp(a)
    return e / e.sum(axis=axis, keepdims=True)


def _dense_attention_unique(x, table, L, pe=None):
    """Independent brute force: ordinary dense multi-head attention over the UNIQUE members of each set."""
    n, C = x.shape
    h = L["heads"]
    d = C // h
    Wq, Wk, Wv = (np.asarray(L["W_qkv"], dtype=np.float64)[i * C:(i + 1) * C] for i in range(3))
    b = np.asarray(L["b_qkv"], dtype=np.float64)
    out = np.zeros((n, C))
    for row in table:
        members = []
        for v in row.tolist():  # order-preserving de-duplication
            if v not in members:
                members.append(v)
        X = x[members]
        Xp = X if pe is None else X + pe[members]
        Q = Xp @ Wq.T + b[:C]
        K = Xp @ Wk.T + b[C:2 * C]
        V = X @ Wv.T + b[2 * C:]
        Y = np.zeros_like(Q)
        for hh in range(h):
            sl = slice(hh * d, (hh + 1) * d)
            A = _softmax(Q[:, sl] @ K[:, sl].T / np.sqrt(d))
            Y[:, sl] = A @ V[:, sl]
        out[members] = Y @ np.asarray(L["W_o"], dtype=np.float64).T + np.asarray(L["b_o"], dtype=np.float64)
    return out


@pytest.mark.parametrize("seed,n,grid,window,tau,C,heads", [
    (1, 150, (16, 16, 1), (6, 6, 1), 5, 16, 4),
    (2, 200, (10, 10, 4), (5, 5, 4), 36, 24, 8),
    (3, 90, (12, 12, 1), (12, 12, 1), 36, 32, 2),
])
def test_masked_duplicates_equal_dense_attention_over_unique_members(oracle, seed, n, grid, window, tau, C, heads):
    cfg = di.random_case(seed, n, grid, window, tau, C, heads)
    x = cfg["feats"].astype(np.float64)
    L = cfg["blocks"][0][0]
    for axis in (0, 1):
        p = oracle.partition(cfg["coords"], 1, grid, window, tau, axis)
        got, covered = oracle.set_attention(x, p.set_table, L["W_qkv"], L["b_qkv"], L["W_o"], L["b_o"], heads)
        assert covered.all()
        want = _dense_attention_unique(x, p.set_table, L)
        assert np.abs(got - want).max() < 1e-12


def test_positional_term_enters_q_and_k_only(oracle):
    cfg = di.random_case(11, 120, (14, 14, 1), (7, 7, 1), 9, 16, 4)
    x = cfg["feats"].astype(np.float64)
    rng = np.random.default_rng(5)
    pe = rng.standard_normal(x.shape)
    L = cfg["blocks"][0][0]
    p = oracle.partition(cfg["coords"], 1, cfg["grid"], cfg["window"], 9, 0)
    got, _ = oracle.set_attention(x, p.set_table, L["W_qkv"], L["b_qkv"], L["W_o"], L["b_o"], 4, pe=pe)
    want = _dense_attention_unique(x, p.set_table, L, pe=pe)
    assert np.abs(got - want).max() < 1e-12
    none, _ = oracle.set_attention(x, p.set_table, L["W_qkv"], L["b_qkv"], L["W_o"], L["b_o"], 4)
    assert np.abs(got - none).max() > 1e-3


def test_full_set_equals_torch_multi_head_attention(oracle):
    """A window with exactly tau voxels has no duplicates: the set attention is textbook MHA."""
    tau, C, heads = 12, 24, 4
    rng = np.random.default_rng(21)
    L = di.make_layer(rng, C, heads, 0, False, False)
    x = rng.standard_normal((tau, C))
    table = np.arange(tau, dtype=np.int32)[None, :]
    got, _ = oracle.set_attention(x, table, L["W_qkv"], L["b_qkv"], L["W_o"], L["b_o"], heads)
    t = lambda a: torch.tensor(np.asarray(a, dtype=np.float64))
    want, _ = torch.nn.functional.multi_head_attention_forward(
        t(x)[:, None, :], t(x)[:, None, :], t(x)[:, None, :], C, heads, t(L["W_qkv"]), t(L["b_qkv"]),
        None, None, False, 0.0, t(L["W_o"]), t(L["b_o"]), need_weights=False)
    assert np.abs(got - want[:, 0, :].numpy()).max() < 1e-12


def test_layer_equals_torch_post_norm_encoder_layer(oracle):
    """MHSA, residual, LN, 2-layer GELU MLP, residual, LN == torch's post-norm TransformerEncoderLayer."""
    tau, C, heads, hidden = 10, 32, 4, 64
    rng = np.random.default_rng(33)
    L = di.make_layer(rng, C, heads, hidden, True, False)
    x = rng.standard_normal((3 * tau, C))
    table = np.arange(3 * tau, dtype=np.int32).reshape(3, tau)  # three full sets
    got = oracle.layer(x, table, L)
    enc = torch.nn.TransformerEncoderLayer(C, heads, hidden, dropout=0.0, activation="gelu", norm_first=False,
                                           layer_norm_eps=1e-5, batch_first=True).double()
    t = lambda a: torch.tensor(np.asarray(a, dtype=np.float64))
    with torch.no_grad():
        enc.self_attn.in_proj_weight.copy_(t(L["W_qkv"])); enc.self_attn.in_proj_bias.copy_(t(L["b_qkv"]))
        enc.self_attn.out_proj.weight.copy_(t(L["W_o"])); enc.self_attn.out_proj.bias.copy_(t(L["b_o"]))
        enc.linear1.weight.copy_(t(L["W_1"])); enc.linear1.bias.copy_(t(L["b_1"]))
        enc.linear2.weight.copy_(t(L["W_2"])); enc.linear2.bias.copy_(t(L["b_2"]))
        enc.norm1.weight.copy_(t(L["ln1_g"])); enc.norm1.bias.copy_(t(L["ln1_b"]))
        enc.norm2.weight.copy_(t(L["ln2_g"])); enc.norm2.bias.copy_(t(L["ln2_b"]))
        enc.train()  # keep the plain (non-fused) path; dropout is 0
        want = enc(t(x).reshape(3, tau, C)).reshape(3 * tau, C).numpy()
    assert np.abs(got - want).max() < 1e-11


def test_closed_form_single_voxel_window(oracle):
    """N = 1: every slot is the same voxel, all but slot 0 masked: Z = W_o (W_v x + b_v) + b_o."""
    C, heads, tau = 16, 4, 6
    rng = np.random.default_rng(8)
    L = di.make_layer(rng, C, heads, 0, False, False)
    x = rng.standard_normal((3, C))
    table = np.array([[1] * tau], dtype=np.int32)
    out = np.full((3, C), 7.0)
    got, covered = oracle.set_attention(x, table, L["W_qkv"], L["b_qkv"], L["W_o"], L["b_o"], heads, out=out)
    W = L["W_qkv"].astype(np.float64)
    want = L["W_o"].astype(np.float64) @ (W[2 * C:] @ x[1] + L["b_qkv"][2 * C:]) + L["b_o"]
    assert np.abs(got[1] - want).max() < 1e-13
    assert list(covered) == [0, 1, 0] and np.all(got[0] == 7.0) and np.all(got[2] == 7.0)  # untouched rows


def test_closed_form_zero_query_gives_mean_of_values(oracle):
    """W_q = 0, b_q = 0: all logits are 0, softmax is uniform over the UNIQUE members."""
    C, heads, tau = 16, 2, 8
    rng = np.random.default_rng(9)
    L = di.make_layer(rng, C, heads, 0, False, False)
    Wqkv = L["W_qkv"].astype(np.float64).copy(); Wqkv[:C] = 0.0
    b = L["b_qkv"].astype(np.float64).copy(); b[:C] = 0.0
    x = rng.standard_normal((5, C))
    table = np.array([[0, 0, 0, 1, 2, 2, 3, 4]], dtype=np.int32)  # duplicates of 0 and 2 are masked
    got, _ = oracle.set_attention(x, table, Wqkv, b, L["W_o"], L["b_o"], heads)
    V = x @ Wqkv[2 * C:].T + b[2 * C:]
    want = L["W_o"].astype(np.float64) @ V.mean(axis=0) + L["b_o"]
    for v in range(5):
        assert np.abs(got[v] - want).max() < 1e-13


def test_layer_without_mlp_and_layernorm_is_residual_attention(oracle):
    cfg = di.random_case(4, 100, (12, 12, 1), (6, 6, 1), 7, 16, 4)
    x = cfg["feats"].astype(np.float64)
    L = cfg["blocks"][0][0]
    p = oracle.partition(cfg["coords"], 1, cfg["grid"], cfg["window"], 7, 0)
    z, _ = oracle.set_attention(x, p.set_table, L["W_qkv"], L["b_qkv"], L["W_o"], L["b_o"], 4)
    assert np.abs(oracle.layer(x, p.set_table, L) - (x + z)).max() < 1e-14


def test_layernorm_and_gelu_against_torch(oracle):
    """A layer whose attention and MLP weights are zero reduces to LN2(LN1(x + b_o) + b_2); with W_1 = I
    scaled into the GELU argument the MLP path exposes GELU itself."""
    C, heads = 8, 2
    rng = np.random.default_rng(12)
    L = di.make_layer(rng, C, heads, C, True, False)
    for k in ("W_qkv", "W_o", "b_qkv", "b_o"):
        L[k] = np.zeros_like(L[k])
    L["W_1"] = np.eye(C, dtype=np.float32) * 2.0
    L["W_2"] = np.eye(C, dtype=np.float32)
    x = rng.standard_normal((6, C)) * 3
    table = np.arange(6, dtype=np.int32).reshape(2, 3)
    got = oracle.layer(x, table, L)
    t = lambda a: torch.tensor(np.asarray(a, dtype=np.float64))
    F = torch.nn.functional
    x1 = F.layer_norm(t(x), (C,), t(L["ln1_g"]), t(L["ln1_b"]), 1e-5)
    m = F.gelu(2.0 * x1 + t(L["b_1"])) + t(L["b_2"])
    want = F.layer_norm(x1 + m, (C,), t(L["ln2_g"]), t(L["ln2_b"]), 1e-5).numpy()
    assert np.abs(got - want).max() < 1e-12


def test_block_is_x_layer_then_y_layer_and_is_window_local(oracle):
    cfg = di.random_case(6, 260, (24, 24, 1), (12, 12, 1), 36, 16, 4, hidden=32, layernorm=True)
    x = cfg["feats"].astype(np.float64)
    coords, grid, window = cfg["coords"], cfg["grid"], cfg["window"]
    Ls = cfg["blocks"][0]
    p0 = oracle.partition(coords, 1, grid, window, 36, 0)
    p1 = oracle.partition(coords, 1, grid, window, 36, 1)
    y = oracle.block(x, p0.set_table, p1.set_table, Ls)
    y2 = oracle.layer(oracle.layer(x, p0.set_table, Ls[0]), p1.set_table, Ls[1])
    assert np.array_equal(y, y2)
    # swapping the two tables changes the result (the rotation matters)
    assert np.abs(oracle.block(x, p1.set_table, p0.set_table, Ls) - y).max() > 1e-3
    # window-local: the block restricted to one window's voxels gives the same rows
    wid = (coords[:, 1] // 12) * 2 + coords[:, 2] // 12
    sel = np.flatnonzero(wid == 3)
    q0 = oracle.partition(coords[sel], 1, grid, window, 36, 0)
    q1 = oracle.partition(coords[sel], 1, grid, window, 36, 1)
    ys = oracle.block(x[sel], q0.set_table, q1.set_table, Ls)
    assert np.abs(ys - y[sel]).max() < 1e-12


def test_threads_do_not_change_results(oracle):
    cfg = di.random_case(14, 300, (24, 24, 1), (12, 12, 1), 36, 16, 4, hidden=32, layernorm=True)
    x = cfg["feats"].astype(np.float64)
    p0 = oracle.partition(cfg["coords"], 1, cfg["grid"], cfg["window"], 36, 0)
    oracle.set_threads(1)
    a = oracle.layer(x, p0.set_table, cfg["blocks"][0][0])
    oracle.set_threads(4)
    b = oracle.layer(x, p0.set_table, cfg["blocks"][0][0])
    assert np.array_equal(a, b)
