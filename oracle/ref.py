"""ctypes access to the CPU oracle (oracle/dsvt_ref.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA library never imports this module and
this module never imports the CUDA library.

Every function takes and returns numpy arrays on the host; features and weights
are float64 (a float32 input is widened exactly).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dsvt_ref.c")
_LIB = os.path.join(_HERE, "libdsvt_ref.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP over independent sets only)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off", _SRC, "-o", tmp, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.dsvt_ref_num_sets.restype = C.c_int64
        _lib.dsvt_ref_num_sets.argtypes = [C.c_int64, C.c_int64]
    return _lib


def _p(a, ct):
    return None if a is None else a.ctypes.data_as(C.POINTER(ct))


def _f64(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float64)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def set_threads(t: int) -> None:
    lib().dsvt_ref_set_threads(int(t))


def max_threads() -> int:
    return int(lib().dsvt_ref_max_threads())


def num_sets(N: int, tau: int) -> int:
    """Eq. 2."""
    return int(lib().dsvt_ref_num_sets(N, tau))


def set_indices(N: int, tau: int) -> np.ndarray:
    """Eq. 3 for one window with N voxels: array [S, tau] of inner-window ranks."""
    S = num_sets(N, tau)
    q = np.zeros((S, tau), dtype=np.int64)
    rc = lib().dsvt_ref_set_indices(C.c_int64(N), C.c_int64(tau), _p(q, C.c_int64))
    if rc != 0:
        raise ValueError("dsvt_ref_set_indices rc=%d" % rc)
    return q


@dataclass
class Partition:
    set_table: np.ndarray  # [S, tau] int32
    perm: np.ndarray  # [n] int32
    win_start: np.ndarray  # [num_windows + 1]
    win_count: np.ndarray  # [num_windows]
    win_setoff: np.ndarray  # [num_windows + 1]

    @property
    def num_sets(self) -> int:
        return int(self.set_table.shape[0])


def num_windows(batch, grid, window, shift=(0, 0, 0)) -> int:
    return int(batch) * int(np.prod([-(-(int(g) + int(s)) // int(w)) for g, w, s in zip(grid, window, shift)]))


def partition(coords, batch, grid, window, set_size, axis, cap_sets: Optional[int] = None,
              shift=(0, 0, 0)) -> Partition:
    """Set partition for one sort axis; `shift` displaces the window cut (hybrid window partition, Sec. 3.2)."""
    coords = _i32(coords).reshape(-1, 4)
    n = coords.shape[0]
    nw = num_windows(batch, grid, window, shift)
    cap = int(cap_sets) if cap_sets is not None else max(n, 1)
    table = np.full((cap, set_size), -1, dtype=np.int32)
    ns = np.zeros(1, dtype=np.int32)
    perm = np.zeros(max(n, 1), dtype=np.int32)
    ws = np.zeros(nw + 1, dtype=np.int32)
    wc = np.zeros(nw + 1, dtype=np.int32)
    wo = np.zeros(nw + 1, dtype=np.int32)
    g = _i32(grid)
    w = _i32(window)
    sh = _i32(shift)
    rc = lib().dsvt_ref_partition_shifted(
        _p(coords, C.c_int32), C.c_int32(n), C.c_int32(batch), _p(g, C.c_int32), _p(w, C.c_int32), _p(sh, C.c_int32),
        C.c_int32(set_size), C.c_int32(axis), _p(table, C.c_int32), C.c_int32(cap), _p(ns, C.c_int32),
        _p(perm, C.c_int32), _p(ws, C.c_int32), _p(wc, C.c_int32), _p(wo, C.c_int32),
    )
    if rc != 0:
        raise ValueError("dsvt_ref_partition_shifted rc=%d" % rc)
    return Partition(table[: ns[0]].copy(), perm[:n].copy(), ws, wc[:nw].copy(), wo)


def rel_bias_len(extent) -> int:
    """Entries per head of a relative position bias table for windows of extent (L, W, H)."""
    L, W, H = (int(v) for v in extent)
    return (2 * L - 1) * (2 * W - 1) * (2 * H - 1)


def set_attention(feats, set_table, W_qkv, b_qkv, W_o, b_o, heads, pe=None, out=None, rpb=None, coords=None,
                  rpb_extent=None):
    """Returns (out [n, C] float64, covered [n] int32).

    rpb: optional relative position bias [heads, rel_bias_len(rpb_extent)], added to the scaled logits and indexed
    by coords[query] - coords[key]; needs coords [n, 4] and rpb_extent = (L, W, H)."""
    feats = _f64(feats)
    n, Cc = feats.shape
    table = _i32(set_table)
    S, tau = table.shape if table.size else (0, table.shape[1] if table.ndim == 2 else 1)
    out = np.zeros((n, Cc), dtype=np.float64) if out is None else out
    covered = np.zeros(max(n, 1), dtype=np.int32)
    Wq, bq, Wo, bo, pe = _f64(W_qkv), _f64(b_qkv), _f64(W_o), _f64(b_o), _f64(pe)
    rpb = _f64(rpb)
    cc = None if rpb is None else _i32(coords).reshape(-1, 4)
    ext = None if rpb is None else _i32(rpb_extent)
    if rpb is not None and rpb.shape != (heads, rel_bias_len(ext)):
        raise ValueError("rpb must be [heads, (2L-1)(2W-1)(2H-1)]")
    rc = lib().dsvt_ref_set_attention_rpb(
        _p(feats, C.c_double), C.c_int32(n), C.c_int32(Cc), _p(table, C.c_int32), C.c_int32(S), C.c_int32(tau),
        _p(Wq, C.c_double), _p(bq, C.c_double), _p(Wo, C.c_double), _p(bo, C.c_double), C.c_int32(heads),
        _p(pe, C.c_double), _p(rpb, C.c_double), _p(cc, C.c_int32), _p(ext, C.c_int32), _p(out, C.c_double),
        _p(covered, C.c_int32),
    )
    if rc != 0:
        raise ValueError("dsvt_ref_set_attention_rpb rc=%d" % rc)
    return out, covered[:n]


class _LayerParams(C.Structure):
    _fields_ = [
        ("C", C.c_int32), ("heads", C.c_int32), ("hidden", C.c_int32), ("set_size", C.c_int32),
        ("ln_eps", C.c_double),
        ("W_qkv", C.POINTER(C.c_double)), ("b_qkv", C.POINTER(C.c_double)),
        ("W_o", C.POINTER(C.c_double)), ("b_o", C.POINTER(C.c_double)),
        ("W_1", C.POINTER(C.c_double)), ("b_1", C.POINTER(C.c_double)),
        ("W_2", C.POINTER(C.c_double)), ("b_2", C.POINTER(C.c_double)),
        ("ln1_g", C.POINTER(C.c_double)), ("ln1_b", C.POINTER(C.c_double)),
        ("ln2_g", C.POINTER(C.c_double)), ("ln2_b", C.POINTER(C.c_double)),
        ("pe", C.POINTER(C.c_double)),
        ("rpb", C.POINTER(C.c_double)), ("coords", C.POINTER(C.c_int32)), ("rpb_extent", C.c_int32 * 3),
    ]


_WEIGHT_KEYS = ["W_qkv", "b_qkv", "W_o", "b_o", "W_1", "b_1", "W_2", "b_2", "ln1_g", "ln1_b", "ln2_g", "ln2_b"]


def _pack_layer(layer: dict, set_size: int, pe=None, coords=None):
    """layer: dict with C, heads, hidden, ln_eps and the arrays of _WEIGHT_KEYS (None allowed); optional "rpb"
    [heads, rel_bias_len(rpb_extent)] with "rpb_extent" = (L, W, H), which needs coords [n, 4]."""
    keep = {}
    p = _LayerParams()
    p.C, p.heads, p.hidden, p.set_size = int(layer["C"]), int(layer["heads"]), int(layer.get("hidden", 0)), int(set_size)
    p.ln_eps = float(layer.get("ln_eps", 1e-5))
    for k in _WEIGHT_KEYS:
        a = _f64(layer.get(k))
        keep[k] = a
        setattr(p, k, _p(a, C.c_double))
    keep["pe"] = _f64(pe)
    p.pe = _p(keep["pe"], C.c_double)
    keep["rpb"] = _f64(layer.get("rpb"))
    if keep["rpb"] is not None:
        if coords is None:
            raise ValueError("a layer with a relative position bias needs coords")
        ext = [int(v) for v in layer["rpb_extent"]]
        if keep["rpb"].shape != (p.heads, rel_bias_len(ext)):
            raise ValueError("rpb must be [heads, (2L-1)(2W-1)(2H-1)]")
        keep["coords"] = _i32(coords).reshape(-1, 4)
        p.rpb = _p(keep["rpb"], C.c_double)
        p.coords = _p(keep["coords"], C.c_int32)
        p.rpb_extent = (C.c_int32 * 3)(*ext)
    return p, keep


def layer(x, set_table, layer_params: dict, pe=None, coords=None):
    x = _f64(x)
    n, Cc = x.shape
    table = _i32(set_table)
    p, keep = _pack_layer(layer_params, table.shape[1], pe, coords)
    y = np.zeros_like(x)
    rc = lib().dsvt_ref_layer(_p(x, C.c_double), C.c_int32(n), _p(table, C.c_int32), C.c_int32(table.shape[0]),
                              C.byref(p), _p(y, C.c_double))
    if rc != 0:
        raise ValueError("dsvt_ref_layer rc=%d" % rc)
    return y


def block(x, table0, table1, layers, pe=None, coords=None):
    """layers: sequence of two layer dicts (X-axis layer, Y-axis layer)."""
    x = _f64(x)
    n, Cc = x.shape
    t0, t1 = _i32(table0), _i32(table1)
    arr = (_LayerParams * 2)()
    keeps = []
    for i in range(2):
        p, keep = _pack_layer(layers[i], t0.shape[1], pe, coords)
        arr[i] = p
        keeps.append(keep)
    y = np.zeros_like(x)
    rc = lib().dsvt_ref_block(_p(x, C.c_double), C.c_int32(n), _p(t0, C.c_int32), C.c_int32(t0.shape[0]),
                              _p(t1, C.c_int32), C.c_int32(t1.shape[0]), arr, _p(y, C.c_double))
    if rc != 0:
        raise ValueError("dsvt_ref_block rc=%d" % rc)
    return y


@dataclass
class Pooled:
    coords: np.ndarray  # [m, 4] int32
    feats: np.ndarray  # [m, C] float64
    region_of: np.ndarray  # [n] int32
    slot_of: np.ndarray  # [n] int32


def pool(coords, feats, batch, grid, pool_shape, W_q, W_k, W_v, W_o, b_q, b_k, b_v, b_o, heads,
         slot_pe=None, mask_empty=0) -> Pooled:
    coords = _i32(coords).reshape(-1, 4)
    feats = _f64(feats)
    n, Cc = feats.shape
    oc = np.zeros((max(n, 1), 4), dtype=np.int32)
    of = np.zeros((max(n, 1), Cc), dtype=np.float64)
    m = np.zeros(1, dtype=np.int32)
    reg = np.zeros(max(n, 1), dtype=np.int32)
    slot = np.zeros(max(n, 1), dtype=np.int32)
    g, pl = _i32(grid), _i32(pool_shape)
    ws = [_f64(a) for a in (W_q, W_k, W_v, W_o, b_q, b_k, b_v, b_o, slot_pe)]
    rc = lib().dsvt_ref_pool(
        _p(coords, C.c_int32), _p(feats, C.c_double), C.c_int32(n), C.c_int32(Cc), C.c_int32(batch),
        _p(g, C.c_int32), _p(pl, C.c_int32), *[_p(a, C.c_double) for a in ws], C.c_int32(heads),
        C.c_int32(mask_empty), _p(oc, C.c_int32), _p(of, C.c_double), C.c_int32(max(n, 1)), _p(m, C.c_int32),
        _p(reg, C.c_int32), _p(slot, C.c_int32),
    )
    if rc != 0:
        raise ValueError("dsvt_ref_pool rc=%d" % rc)
    return Pooled(oc[: m[0]].copy(), of[: m[0]].copy(), reg[:n].copy(), slot[:n].copy())


def bev_scatter(coords, feats, batch, grid, channels_last=False) -> np.ndarray:
    """Dense bird's-eye-view map: [batch, C*Z, Y, X] (or [batch, Y, X, C*Z] when channels_last), zeros where no voxel."""
    coords = _i32(coords).reshape(-1, 4)
    feats = _f64(feats)
    n, Cc = feats.shape
    g = _i32(grid)
    X, Y, Z = (int(v) for v in g)
    shape = (batch, Y, X, Cc * Z) if channels_last else (batch, Cc * Z, Y, X)
    out = np.empty(shape, dtype=np.float64)
    rc = lib().dsvt_ref_bev_scatter(_p(coords, C.c_int32), _p(feats, C.c_double), C.c_int32(n), C.c_int32(Cc),
                                    C.c_int32(batch), _p(g, C.c_int32), C.c_int32(1 if channels_last else 0),
                                    _p(out, C.c_double))
    if rc != 0:
        raise ValueError("dsvt_ref_bev_scatter rc=%d" % rc)
    return out
