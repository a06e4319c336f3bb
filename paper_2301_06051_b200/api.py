"""Thin ctypes binding of the C ABI in include/dsvt.h.

Argument marshalling only: every step of the path runs in the CUDA library.  torch supplies device
memory (tensor.data_ptr()) and the stream.  There is no CPU fallback: if the shared library is
missing, loading raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Dict, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdsvt_b200.so")

OK = 0
FP32 = 0
BF16_FP32ACC = 1
STATUS_BAD_COORD, STATUS_TABLE_OVERFLOW, STATUS_BAD_INDEX, STATUS_DUPLICATE_CELL, STATUS_TIMEOUT = 1, 2, 4, 8, 16

EXPORTS = [
    "dsvt_create", "dsvt_destroy", "dsvt_status_sync", "dsvt_last_cuda_error", "dsvt_error_string",
    "dsvt_launch_count", "dsvt_set_layer_ctas", "dsvt_partition", "dsvt_partition_rotated", "dsvt_partition_shifted", "dsvt_partition_counted", "dsvt_pool_counted", "dsvt_partition_noalloc", "dsvt_set_attention", "dsvt_set_attention_rpb", "dsvt_layer", "dsvt_layers", "dsvt_block", "dsvt_pool",
    "dsvt_bev_scatter", "dsvt_fma_probe",
]

_lib = None


class DsvtError(RuntimeError):
    def __init__(self, code: int, where: str, cuda: int = 0):
        self.code = code
        msg = load().dsvt_error_string(code).decode()
        super().__init__("%s: %s (code %d%s)" % (where, msg, code, ", cudaError %d" % cuda if cuda else ""))


class LayerParams(C.Structure):
    """Mirror of dsvt_layer_params."""
    _fields_ = [
        ("C", C.c_int32), ("heads", C.c_int32), ("hidden", C.c_int32), ("set_size", C.c_int32),
        ("precision", C.c_int32), ("ln_eps", C.c_float),
        ("W_qkv", C.c_void_p), ("W_o", C.c_void_p), ("W_1", C.c_void_p), ("W_2", C.c_void_p),
        ("b_qkv", C.c_void_p), ("b_o", C.c_void_p), ("b_1", C.c_void_p), ("b_2", C.c_void_p),
        ("ln1_g", C.c_void_p), ("ln1_b", C.c_void_p), ("ln2_g", C.c_void_p), ("ln2_b", C.c_void_p),
        ("pe", C.c_void_p),
        ("rpb", C.c_void_p), ("coords", C.c_void_p), ("rpb_extent", C.c_int32 * 3),
    ]


class TableRef(C.Structure):
    """Mirror of dsvt_table_ref."""
    _fields_ = [("set_table", C.c_void_p), ("cap_sets", C.c_int32), ("num_sets", C.c_void_p),
                ("set_rowoff", C.c_void_p)]


MAX_CHAIN_LAYERS = 16


def load():
    """Loads the CUDA library (built by paper_2301_06051_b200.build); raises if it is absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError("%s is missing: run `python -m paper_2301_06051_b200.build` (needs nvcc)" % LIB_PATH)
    lib = C.CDLL(LIB_PATH)
    i32, i64, vp = C.c_int32, C.c_int64, C.c_void_p
    p3 = C.POINTER(C.c_int32)
    lib.dsvt_create.argtypes = [C.POINTER(vp), C.c_int, vp, i64, i64, i32]
    lib.dsvt_destroy.argtypes = [vp]
    lib.dsvt_status_sync.argtypes = [vp, C.POINTER(i32)]
    lib.dsvt_last_cuda_error.argtypes = [vp]
    lib.dsvt_error_string.argtypes = [C.c_int]
    lib.dsvt_error_string.restype = C.c_char_p
    lib.dsvt_launch_count.argtypes = [vp]
    lib.dsvt_launch_count.restype = i64
    lib.dsvt_set_layer_ctas.argtypes = [vp, i32]
    lib.dsvt_partition.argtypes = [vp, vp, i32, i32, p3, p3, i32, i32, vp, i32, vp, vp, vp, vp, vp, vp]
    lib.dsvt_partition_rotated.argtypes = [vp, vp, i32, i32, p3, p3, i32, vp, i32, vp, vp, vp, vp, vp, vp]
    lib.dsvt_partition_shifted.argtypes = [vp, vp, i32, i32, p3, p3, p3, i32, vp, i32, vp, vp, vp, vp, vp, vp]
    lib.dsvt_partition_counted.argtypes = [vp, vp, i32, vp, i32, p3, p3, p3, i32, vp, i32, vp, vp, vp, vp, vp, vp]
    lib.dsvt_pool_counted.argtypes = [vp, vp, vp, i32, vp, i32, i32, p3, p3, vp, vp, vp, vp, vp, vp, vp, vp, vp, i32,
                                      i32, C.c_int, vp, vp, i32, vp, vp, vp]
    lib.dsvt_partition_noalloc.argtypes = [vp, vp, i32, i32, p3, p3, i32, i32, vp, i32, vp, vp, vp, C.POINTER(i32)]
    lib.dsvt_set_attention.argtypes = [vp, vp, i32, i32, vp, i32, vp, vp, i32, vp, vp, vp, vp, i32, vp, C.c_int, vp]
    lib.dsvt_set_attention_rpb.argtypes = [vp, vp, i32, i32, vp, i32, vp, vp, i32, vp, vp, vp, vp, i32, vp, vp, vp, p3,
                                           C.c_int, vp]
    lib.dsvt_bev_scatter.argtypes = [vp, vp, vp, i32, i32, i32, p3, i32, vp]
    lib.dsvt_layer.argtypes = [vp, vp, i32, vp, i32, vp, vp, C.POINTER(LayerParams), vp]
    lib.dsvt_fma_probe.argtypes = [vp, i32, i32, i32, vp, C.POINTER(i64)]
    lib.dsvt_layers.argtypes = [vp, vp, i32, i32, C.POINTER(TableRef), C.POINTER(LayerParams), vp]
    lib.dsvt_block.argtypes = [vp, vp, i32, vp, i32, vp, vp, vp, i32, vp, vp, C.POINTER(LayerParams), vp]
    lib.dsvt_pool.argtypes = [vp, vp, vp, i32, i32, i32, p3, p3, vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, i32,
                              C.c_int, vp, vp, i32, vp, vp, vp]
    for name in EXPORTS:
        if name not in ("dsvt_error_string", "dsvt_launch_count"):
            getattr(lib, name).restype = C.c_int
    _lib = lib
    return lib


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device-resident contiguous tensors only"
    return t.data_ptr()


def _i3(v: Sequence[int]):
    return (C.c_int32 * 3)(int(v[0]), int(v[1]), int(v[2]))


def device_weights(layer: Dict, precision: int, device) -> Dict:
    """Moves one layer's numpy parameters (see dsvt_inputs.make_layer) to the device in the storage
    the chosen precision expects: matrices float32 or bfloat16, everything else float32."""
    import numpy as np

    out: Dict = {k: layer[k] for k in ("C", "heads", "hidden", "rpb_extent") if k in layer}
    out["ln_eps"] = float(layer.get("ln_eps", 1e-5))
    out["precision"] = precision
    for k, v in layer.items():
        if not isinstance(v, np.ndarray):
            continue
        t = torch.from_numpy(np.ascontiguousarray(v, dtype=np.float32)).to(device)
        if k.startswith("W_") and precision == BF16_FP32ACC:
            tb = t.to(torch.bfloat16)
            assert torch.equal(tb.float(), t), "bfloat16 precision needs bfloat16-representable weights"
            t = tb
        out[k] = t.contiguous()
    return out


def layer_params(w: Dict, set_size: int, pe: Optional[torch.Tensor] = None,
                 coords: Optional[torch.Tensor] = None) -> LayerParams:
    """w may hold "rpb" (float tensor [heads, (2L-1)(2W-1)(2H-1)]) and "rpb_extent" = (L, W, H); then coords
    (int32 [n, 4]) is required."""
    p = LayerParams()
    p.C, p.heads, p.hidden, p.set_size = int(w["C"]), int(w["heads"]), int(w.get("hidden", 0)), int(set_size)
    p.precision = int(w["precision"])
    p.ln_eps = float(w.get("ln_eps", 1e-5))
    for k in ("W_qkv", "W_o", "W_1", "W_2", "b_qkv", "b_o", "b_1", "b_2", "ln1_g", "ln1_b", "ln2_g", "ln2_b"):
        setattr(p, k, _ptr(w.get(k)))
    p.pe = _ptr(pe)
    if w.get("rpb") is not None:
        if coords is None:
            raise ValueError("a layer with a relative position bias needs coords")
        p.rpb = _ptr(w["rpb"])
        p.coords = _ptr(coords)
        p.rpb_extent = _i3(w["rpb_extent"])
    return p


@dataclass
class SetTable:
    """Device-side result of dsvt_partition."""
    set_table: torch.Tensor  # int32 [cap_sets, set_size]
    num_sets: torch.Tensor  # int32 [1] (device)
    set_rowoff: torch.Tensor  # int32 [4 * cap_sets + 4]: row offsets, then the tile plan
    cap_sets: int
    set_size: int
    perm: Optional[torch.Tensor] = None
    win_start: Optional[torch.Tensor] = None
    win_count: Optional[torch.Tensor] = None
    win_setoff: Optional[torch.Tensor] = None


NOALLOC_MAX_VOXELS = 65536
NOALLOC_MAX_WINDOWS = 65536


def partition_noalloc(coords: torch.Tensor, batch: int, grid, window, set_size: int, axis: int, out: SetTable,
                      status_bits: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None) -> SetTable:
    """dsvt_partition_noalloc: the set partition for callers that must not allocate device memory.

    Needs no Context.  `out` (and `status_bits`, a device int32) are the caller's own buffers; the
    library's workspace is a fixed array inside the shared library, so at most NOALLOC_MAX_VOXELS voxels
    and NOALLOC_MAX_WINDOWS windows fit.  Calls that overlap on the GPU race on that array.
    """
    lib = load()
    st = stream if stream is not None else torch.cuda.current_stream(coords.device)
    err = C.c_int32(0)
    with torch.cuda.device(coords.device):
        rc = lib.dsvt_partition_noalloc(C.c_void_p(st.cuda_stream), _ptr(coords), int(coords.shape[0]), int(batch),
                                        _i3(grid), _i3(window), int(set_size), int(axis), _ptr(out.set_table),
                                        out.cap_sets, _ptr(out.num_sets), _ptr(out.set_rowoff), _ptr(status_bits),
                                        C.byref(err))
    if rc != OK:
        raise DsvtError(rc, "dsvt_partition_noalloc", int(err.value))
    return out


class Context:
    """Owns a dsvt_ctx bound to the current torch CUDA stream of `device`."""

    def __init__(self, max_voxels: int, max_windows: int, max_channels: int = 256, device: int = 0,
                 stream: Optional[torch.cuda.Stream] = None):
        self.lib = load()
        if not torch.cuda.is_available():
            raise RuntimeError("the DSVT library needs a CUDA device; there is no CPU path")
        self.device = torch.device("cuda", device)
        self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
        self.limits = (int(max_voxels), int(max_windows), int(max_channels))
        self._h = C.c_void_p()
        rc = self.lib.dsvt_create(C.byref(self._h), device, C.c_void_p(self.stream.cuda_stream), int(max_voxels),
                                  int(max_windows), int(max_channels))
        if rc != OK:
            raise DsvtError(rc, "dsvt_create")

    def sibling(self, stream: torch.cuda.Stream) -> "Context":
        """A second context with the same limits on the same device, bound to `stream` (its own workspace and
        status word: calls on the two contexts may overlap on the GPU)."""
        return Context(*self.limits, device=self.device.index, stream=stream)

    def close(self):
        if self._h:
            self.lib.dsvt_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc: int, where: str):
        if rc != OK:
            raise DsvtError(rc, where, self.lib.dsvt_last_cuda_error(self._h))

    def status_sync(self) -> int:
        """Synchronises and returns (and clears) the device status bits."""
        bits = C.c_int32(0)
        rc = self.lib.dsvt_status_sync(self._h, C.byref(bits))
        if rc not in (OK, -5, -6):
            raise DsvtError(rc, "dsvt_status_sync", self.lib.dsvt_last_cuda_error(self._h))
        return int(bits.value)

    def launch_count(self) -> int:
        return int(self.lib.dsvt_launch_count(self._h))

    def set_layer_ctas(self, max_ctas: int) -> None:
        """Caps the tensor-core layer kernel's persistent CTAs on this context (0: one per SM)."""
        self._check(self.lib.dsvt_set_layer_ctas(self._h, int(max_ctas)), "dsvt_set_layer_ctas")

    # ---- dsvt_partition ----
    def partition(self, coords: torch.Tensor, batch: int, grid, window, set_size: int, axis: int,
                  cap_sets: Optional[int] = None, extras: bool = False, out: Optional[SetTable] = None) -> SetTable:
        n = int(coords.shape[0])
        if out is None:
            cap = int(cap_sets) if cap_sets is not None else max(n, 1)
            dev = self.device
            out = SetTable(torch.empty((cap, set_size), dtype=torch.int32, device=dev),
                           torch.zeros(1, dtype=torch.int32, device=dev),
                           torch.empty(4 * cap + 4, dtype=torch.int32, device=dev), cap, set_size)
            if extras:
                nw = int(batch) * (-(-grid[0] // window[0])) * (-(-grid[1] // window[1])) * (-(-grid[2] // window[2]))
                out.perm = torch.empty(max(n, 1), dtype=torch.int32, device=dev)
                out.win_start = torch.empty(nw + 1, dtype=torch.int32, device=dev)
                out.win_count = torch.empty(nw, dtype=torch.int32, device=dev)
                out.win_setoff = torch.empty(nw + 1, dtype=torch.int32, device=dev)
        rc = self.lib.dsvt_partition(self._h, _ptr(coords), n, int(batch), _i3(grid), _i3(window), int(set_size),
                                     int(axis), _ptr(out.set_table), out.cap_sets, _ptr(out.num_sets),
                                     _ptr(out.set_rowoff), _ptr(out.perm), _ptr(out.win_start), _ptr(out.win_count),
                                     _ptr(out.win_setoff))
        self._check(rc, "dsvt_partition")
        return out

    # ---- dsvt_partition_rotated ----
    def partition_rotated(self, coords: torch.Tensor, batch: int, grid, window, set_size: int,
                          cap_sets: Optional[int] = None, out=None, shift=None, n_dev: Optional[torch.Tensor] = None):
        """Both sort axes in one call; returns (X-axis SetTable, Y-axis SetTable).  `shift` displaces the window
        cut (dsvt_partition_shifted); None calls dsvt_partition_rotated.  `n_dev` (device int32) gives the voxel
        count where it lives on the device (dsvt_partition_counted); coords' length is then the capacity."""
        n = int(coords.shape[0])
        if out is None:
            cap = int(cap_sets) if cap_sets is not None else max(n, 1)
            dev = self.device
            out = tuple(SetTable(torch.empty((cap, set_size), dtype=torch.int32, device=dev),
                                 torch.zeros(1, dtype=torch.int32, device=dev),
                                 torch.empty(4 * cap + 4, dtype=torch.int32, device=dev), cap, set_size)
                        for _ in range(2))
        t0, t1 = out
        assert t0.cap_sets == t1.cap_sets and t0.set_size == t1.set_size == set_size
        pair = lambda a, b: (C.c_void_p * 2)(_ptr(a), _ptr(b))
        tail = (int(set_size), pair(t0.set_table, t1.set_table), t0.cap_sets, pair(t0.num_sets, t1.num_sets),
                pair(t0.set_rowoff, t1.set_rowoff), pair(t0.perm, t1.perm), _ptr(t0.win_start), _ptr(t0.win_count),
                _ptr(t0.win_setoff))
        if n_dev is not None:
            rc = self.lib.dsvt_partition_counted(self._h, _ptr(coords), n, _ptr(n_dev), int(batch), _i3(grid),
                                                 _i3(window), None if shift is None else _i3(shift), *tail)
            self._check(rc, "dsvt_partition_counted")
        elif shift is None:
            rc = self.lib.dsvt_partition_rotated(self._h, _ptr(coords), n, int(batch), _i3(grid), _i3(window), *tail)
            self._check(rc, "dsvt_partition_rotated")
        else:
            rc = self.lib.dsvt_partition_shifted(self._h, _ptr(coords), n, int(batch), _i3(grid), _i3(window),
                                                 _i3(shift), *tail)
            self._check(rc, "dsvt_partition_shifted")
        return out

    # ---- dsvt_set_attention ----
    def set_attention(self, feats: torch.Tensor, table: SetTable, w: Dict, out: torch.Tensor,
                      pe: Optional[torch.Tensor] = None, use_rowoff: bool = True,
                      coords: Optional[torch.Tensor] = None) -> torch.Tensor:
        n, Cc = int(feats.shape[0]), int(feats.shape[1])
        if w.get("rpb") is not None:  # dsvt_set_attention_rpb
            rc = self.lib.dsvt_set_attention_rpb(
                self._h, _ptr(feats), n, Cc, _ptr(table.set_table), table.cap_sets, _ptr(table.num_sets),
                _ptr(table.set_rowoff) if use_rowoff else None, table.set_size, _ptr(w["W_qkv"]), _ptr(w.get("b_qkv")),
                _ptr(w["W_o"]), _ptr(w.get("b_o")), int(w["heads"]), _ptr(pe), _ptr(w["rpb"]), _ptr(coords),
                _i3(w["rpb_extent"]), int(w["precision"]), _ptr(out))
            self._check(rc, "dsvt_set_attention_rpb")
            return out
        rc = self.lib.dsvt_set_attention(self._h, _ptr(feats), n, Cc, _ptr(table.set_table), table.cap_sets,
                                         _ptr(table.num_sets), _ptr(table.set_rowoff) if use_rowoff else None,
                                         table.set_size, _ptr(w["W_qkv"]), _ptr(w.get("b_qkv")), _ptr(w["W_o"]),
                                         _ptr(w.get("b_o")), int(w["heads"]), _ptr(pe), int(w["precision"]), _ptr(out))
        self._check(rc, "dsvt_set_attention")
        return out

    # ---- dsvt_layer ----
    def layer(self, x: torch.Tensor, table: SetTable, w: Dict, y: torch.Tensor, pe: Optional[torch.Tensor] = None,
              use_rowoff: bool = True, coords: Optional[torch.Tensor] = None) -> torch.Tensor:
        p = layer_params(w, table.set_size, pe, coords)
        rc = self.lib.dsvt_layer(self._h, _ptr(x), int(x.shape[0]), _ptr(table.set_table), table.cap_sets,
                                 _ptr(table.num_sets), _ptr(table.set_rowoff) if use_rowoff else None, C.byref(p),
                                 _ptr(y))
        self._check(rc, "dsvt_layer")
        return y

    # ---- dsvt_layers ----
    def layers(self, x: torch.Tensor, tables: Sequence["SetTable"], ws: Sequence[Dict], y: torch.Tensor,
               coords: Optional[torch.Tensor] = None, use_rowoff: bool = True,
               pe: Optional[torch.Tensor] = None) -> torch.Tensor:
        """A chain of layers, layer i on tables[i] with weights ws[i]: the first reads x, all write y."""
        L = len(ws)
        assert len(tables) == L
        tr = (TableRef * max(L, 1))()
        pr = (LayerParams * max(L, 1))()
        for i, (t, w) in enumerate(zip(tables, ws)):
            tr[i].set_table, tr[i].cap_sets, tr[i].num_sets = _ptr(t.set_table), t.cap_sets, _ptr(t.num_sets)
            tr[i].set_rowoff = _ptr(t.set_rowoff) if use_rowoff else None
            pr[i] = layer_params(w, t.set_size, pe, coords)
        rc = self.lib.dsvt_layers(self._h, _ptr(x), int(x.shape[0]), L, tr, pr, _ptr(y))
        self._check(rc, "dsvt_layers")
        return y

    # ---- dsvt_block ----
    def block(self, x: torch.Tensor, t0: SetTable, t1: SetTable, ws: Sequence[Dict], y: torch.Tensor,
              pe: Optional[torch.Tensor] = None, coords: Optional[torch.Tensor] = None) -> torch.Tensor:
        arr = (LayerParams * 2)(layer_params(ws[0], t0.set_size, pe, coords),
                                layer_params(ws[1], t1.set_size, pe, coords))
        rc = self.lib.dsvt_block(self._h, _ptr(x), int(x.shape[0]), _ptr(t0.set_table), t0.cap_sets,
                                 _ptr(t0.num_sets), _ptr(t0.set_rowoff), _ptr(t1.set_table), t1.cap_sets,
                                 _ptr(t1.num_sets), _ptr(t1.set_rowoff), arr, _ptr(y))
        self._check(rc, "dsvt_block")
        return y

    # ---- dsvt_fma_probe ----
    def fma_probe(self, blocks: int, threads: int, iters: int, sink: torch.Tensor) -> int:
        """Enqueues the FP32 FMA probe kernel; returns the floating-point operations of the launch."""
        flops = C.c_int64(0)
        rc = self.lib.dsvt_fma_probe(self._h, int(blocks), int(threads), int(iters), _ptr(sink), C.byref(flops))
        self._check(rc, "dsvt_fma_probe")
        return int(flops.value)

    # ---- dsvt_bev_scatter ----
    def bev_scatter(self, coords: torch.Tensor, feats: torch.Tensor, batch: int, grid, channels_last: bool = False,
                    out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """Dense BEV map [batch, C*Z, Y, X] (or [batch, Y, X, C*Z] when channels_last), written in full."""
        n, Cc = int(feats.shape[0]), int(feats.shape[1])
        X, Y, Z = (int(v) for v in grid)
        shape = (batch, Y, X, Cc * Z) if channels_last else (batch, Cc * Z, Y, X)
        if out is None:
            out = torch.empty(shape, dtype=torch.float32, device=self.device)
        assert tuple(out.shape) == shape and out.dtype == torch.float32
        rc = self.lib.dsvt_bev_scatter(self._h, _ptr(coords), _ptr(feats), n, Cc, int(batch), _i3(grid),
                                       1 if channels_last else 0, _ptr(out))
        self._check(rc, "dsvt_bev_scatter")
        return out

    # ---- dsvt_pool ----
    def pool(self, coords: torch.Tensor, feats: torch.Tensor, batch: int, grid, pool_shape, w: Dict,
             mask_empty: int = 0, cap_m: Optional[int] = None, extras: bool = False,
             n_dev: Optional[torch.Tensor] = None):
        """Returns (out_coords [cap_m,4], out_feats [cap_m,C], num_out [1], region_of, slot_of).  `n_dev` (device
        int32): the input's voxel count where it lives on the device (dsvt_pool_counted)."""
        n, Cc = int(feats.shape[0]), int(feats.shape[1])
        cap = int(cap_m) if cap_m is not None else max(n, 1)
        dev = self.device
        oc = torch.empty((cap, 4), dtype=torch.int32, device=dev)
        of = torch.empty((cap, Cc), dtype=torch.float32, device=dev)
        num = torch.zeros(1, dtype=torch.int32, device=dev)
        reg = torch.empty(max(n, 1), dtype=torch.int32, device=dev) if extras else None
        slot = torch.empty(max(n, 1), dtype=torch.int32, device=dev) if extras else None
        tail = (Cc, int(batch), _i3(grid), _i3(pool_shape), _ptr(w["W_q"]), _ptr(w["W_k"]), _ptr(w["W_v"]),
                _ptr(w["W_o"]), _ptr(w.get("b_q")), _ptr(w.get("b_k")), _ptr(w.get("b_v")), _ptr(w.get("b_o")),
                _ptr(w.get("slot_pe")), int(w["heads"]), int(mask_empty), int(w["precision"]), _ptr(oc), _ptr(of), cap,
                _ptr(num), _ptr(reg), _ptr(slot))
        if n_dev is not None:
            rc = self.lib.dsvt_pool_counted(self._h, _ptr(coords), _ptr(feats), n, _ptr(n_dev), *tail)
            self._check(rc, "dsvt_pool_counted")
        else:
            rc = self.lib.dsvt_pool(self._h, _ptr(coords), _ptr(feats), n, *tail)
            self._check(rc, "dsvt_pool")
        return oc, of, num, reg, slot
