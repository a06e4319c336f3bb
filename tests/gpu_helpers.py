"""Shared helpers of the GPU parity tests (marshalling and error metrics only)."""
import numpy as np
import torch

from paper_2301_06051_b200 import api

FP32_ATOL = 1e-4  # fp32 path: max-abs error against the float64 oracle
BF16_RTOL = 2e-2  # bf16-weight path: max|g - r| / max|r| per output tensor


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda().contiguous()


def precision_of(cfg):
    return api.BF16_FP32ACC if cfg["precision"] == "bf16" else api.FP32


def check_close(got, want, cfg_precision, what=""):
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    assert got.shape == want.shape, (what, got.shape, want.shape)
    assert np.all(np.isfinite(got)), what
    err = np.abs(got - want).max() if got.size else 0.0
    if cfg_precision == "bf16":
        rel = err / max(np.abs(want).max() if want.size else 0.0, 1e-6)
        assert rel <= BF16_RTOL, "%s: relative error %.3e > %.1e" % (what, rel, BF16_RTOL)
        return rel
    assert err <= FP32_ATOL, "%s: max-abs error %.3e > %.1e" % (what, err, FP32_ATOL)
    return err


def row_rel_error(got, want) -> float:
    """Largest per-row relative error max_i |g_i - r_i|_inf / |r_i|_inf (reported beside the tensor-wide figure)."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    if got.size == 0:
        return 0.0
    num = np.abs(got - want).max(axis=1)
    den = np.maximum(np.abs(want).max(axis=1), 1e-6)
    return float((num / den).max())


def table_np(t: api.SetTable):
    """(table rows [S, tau], set_rowoff [S + 1]) on the host."""
    S = int(t.num_sets.item())
    return t.set_table[:S].cpu().numpy(), t.set_rowoff[: S + 1].cpu().numpy()


def rowoff_of(table: np.ndarray) -> np.ndarray:
    """Distinct-member offsets implied by a table: slot k counts iff k == 0 or row[k] != row[k-1]."""
    if table.shape[0] == 0:
        return np.zeros(1, dtype=np.int32)
    uniq = np.ones(table.shape, dtype=bool)
    uniq[:, 1:] = table[:, 1:] != table[:, :-1]
    return np.concatenate([[0], np.cumsum(uniq.sum(axis=1))]).astype(np.int32)


def upload_table(table: np.ndarray, with_rowoff=True, cap_extra=0) -> api.SetTable:
    """A caller-made table on the device (optionally without row offsets)."""
    S, tau = table.shape
    cap = S + cap_extra
    full = np.full((max(cap, 1), tau), -7, dtype=np.int32)
    full[:S] = table
    ro = np.zeros(4 * max(cap, 1) + 4, dtype=np.int32)  # row offsets, then "no tile plan"
    ro[: S + 1] = rowoff_of(table)
    ro[(max(cap, 1) if S else 0) + 1] = -1
    return api.SetTable(dev(full), dev(np.array([S], dtype=np.int32)), dev(ro) if with_rowoff else None,
                        max(cap, 1) if S else 0, tau)
