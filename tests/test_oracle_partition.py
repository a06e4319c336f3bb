"""Pins for the oracle's partition (Sec. 3.2, Eq. 1-3, Theorems A.2-A.4). CPU only."""
import os

import numpy as np
import pytest

import dsvt_inputs as di

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _read_eq3():
    cases = []
    for line in open(os.path.join(GOLD, "eq3_rows.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        head, rows = line.split("|")
        N, tau = (int(t) for t in head.split())
        cases.append((N, tau, np.array([[int(t) for t in r.split()] for r in rows.split(";")], dtype=np.int64)))
    return cases


def test_eq3_hand_worked_rows(oracle):
    cases = _read_eq3()
    assert len(cases) >= 5
    for N, tau, want in cases:
        got = oracle.set_indices(N, tau)
        assert got.shape == want.shape, (N, tau)
        assert np.array_equal(got, want), (N, tau, got, want)


def _read_tiny_grid(name="tiny_grid.txt"):
    sect, data = None, {"coords": [], "axis0": [], "axis1": []}
    for line in open(os.path.join(GOLD, name)):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line in data:
            sect = line
            continue
        data[sect].append([int(t) for t in line.split()])
    return {k: np.array(v, dtype=np.int32) for k, v in data.items()}


def test_tiny_grid_hand_worked_tables(oracle):
    g = _read_tiny_grid()
    for axis in (0, 1):
        p = oracle.partition(g["coords"], 1, (8, 4, 1), (4, 4, 1), 3, axis)
        assert np.array_equal(p.set_table, g["axis%d" % axis]), axis
        assert list(p.win_count) == [7, 2]
        assert list(p.win_start) == [0, 7, 9]
        assert list(p.win_setoff) == [0, 3, 4]
    px = oracle.partition(g["coords"], 1, (8, 4, 1), (4, 4, 1), 3, 0).perm
    py = oracle.partition(g["coords"], 1, (8, 4, 1), (4, 4, 1), 3, 1).perm
    assert list(px) == [4, 1, 2, 6, 5, 0, 8, 7, 3]
    assert list(py) == [4, 2, 0, 1, 5, 6, 8, 7, 3]


def test_tiny_grid_shifted_hand_worked_tables(oracle):
    """Window cut displaced by (2, 0, 0): hand-worked tables, counts and orders."""
    g = _read_tiny_grid("tiny_grid_shift.txt")
    for axis in (0, 1):
        p = oracle.partition(g["coords"], 1, (8, 4, 1), (4, 4, 1), 3, axis, shift=(2, 0, 0))
        assert np.array_equal(p.set_table, g["axis%d" % axis]), axis
        assert list(p.win_count) == [4, 5, 0]
        assert list(p.win_start) == [0, 4, 9, 9]
        assert list(p.win_setoff) == [0, 2, 4, 4]
    assert list(oracle.partition(g["coords"], 1, (8, 4, 1), (4, 4, 1), 3, 0, shift=(2, 0, 0)).perm) == [4, 1, 2, 6, 5, 0, 8, 7, 3]
    assert list(oracle.partition(g["coords"], 1, (8, 4, 1), (4, 4, 1), 3, 1, shift=(2, 0, 0)).perm) == [4, 2, 1, 6, 7, 0, 5, 8, 3]


@pytest.mark.parametrize("grid,window,shift,batch,n,tau", [
    ((20, 17, 1), (6, 5, 1), (3, 2, 0), 1, 200, 7),
    ((9, 9, 6), (4, 4, 3), (2, 1, 1), 2, 500, 10),
    ((64, 64, 1), (24, 24, 1), (12, 12, 0), 1, 2000, 36),
])
def test_shifted_partition_is_the_plain_partition_of_translated_voxels(oracle, grid, window, shift, batch, n, tau):
    """Displacing the window cut by s is the same as moving every voxel by +s on a grid that is s cells larger:
    this reduces the shifted partition to the unshifted one, which the tests above pin on its own; also the
    brute-force restatement with the shift written out."""
    rng = np.random.default_rng(11)
    coords = di.unique_cells(rng, n, grid, batch)
    moved = coords.copy()
    moved[:, 1:] += np.array(shift, dtype=np.int32)
    big = tuple(g + s for g, s in zip(grid, shift))
    for axis in (0, 1):
        p = oracle.partition(coords, batch, grid, window, tau, axis, shift=shift)
        q = oracle.partition(moved, batch, big, window, tau, axis)
        assert np.array_equal(p.set_table, q.set_table)
        assert np.array_equal(p.perm, q.perm)
        assert np.array_equal(p.win_count, q.win_count) and np.array_equal(p.win_setoff, q.win_setoff)
        assert np.array_equal(p.set_table, _brute_partition(moved, batch, big, window, tau, axis))
    # a shift of zero is the plain partition; a shift outside [0, window) is refused
    assert np.array_equal(oracle.partition(coords, batch, grid, window, tau, 0, shift=(0, 0, 0)).set_table,
                          oracle.partition(coords, batch, grid, window, tau, 0).set_table)
    with pytest.raises(ValueError):
        oracle.partition(coords, batch, grid, window, tau, 0, shift=(window[0], 0, 0))


@pytest.mark.parametrize("tau", [3, 24, 36, 48, 60, 90])
def test_theorems_a2_a3_a4(oracle, tau):
    """Non-overlap (A.2), completeness (A.3), balanced sizes (A.4), and Eq. 2's minimality."""
    for N in list(range(1, 700)) + [1151, 1152, 1153, 4607, 4608]:
        q = oracle.set_indices(N, tau)
        S = q.shape[0]
        assert S == -(-N // tau)  # fewest sets of capacity tau that cover N
        assert (S - 1) * tau < N <= S * tau
        assert q.min() == 0 and q.max() == N - 1
        assert np.all(np.diff(q.reshape(-1)) >= 0)  # ranks never decrease along (j, k)
        assert np.all(np.diff(q.reshape(-1)) <= 1)  # and never skip a voxel (A.3)
        uniq = [np.unique(r) for r in q]
        allm = np.concatenate(uniq)
        assert allm.shape[0] == N and np.array_equal(np.sort(allm), np.arange(N))  # A.2 + A.3
        sizes = np.array([u.shape[0] for u in uniq])
        assert sizes.min() >= N // S and sizes.max() <= N // S + 1  # A.4
        # first index of set j is floor(j*N/S) (Eq. A.3 in the proof of Theorem A.2)
        assert np.array_equal(q[:, 0], (np.arange(S) * N) // S)
        if N == S * tau:  # the trivial case named in Appendix A: no duplicates at all
            assert np.array_equal(q.reshape(-1), np.arange(N))


def test_eq3_not_float_evaluation(oracle):
    """Exact integer floor: a float evaluation of Eq. 3 is off by one at N=81, tau=36, S=3, m=20."""
    q = oracle.set_indices(81, 36)
    assert q.shape == (3, 36)
    assert q.reshape(-1)[20] == (20 * 81) // (3 * 36) == 15


def _brute_partition(coords, batch, grid, window, tau, axis):
    """Independent restatement with python tuples and sorted()."""
    L, W, H = window
    nW = [-(-grid[a] // window[a]) for a in range(3)]
    wins = {}
    for i, (b, x, y, z) in enumerate(coords.tolist()):
        wid = ((b * nW[0] + x // L) * nW[1] + y // W) * nW[2] + z // H
        xi, yi, zi = x % L, y % W, z % H
        key = (xi, yi, zi) if axis == 0 else (yi, xi, zi)
        wins.setdefault(wid, []).append((key, i))
    rows = []
    for wid in sorted(wins):
        members = [i for _, i in sorted(wins[wid])]
        N = len(members)
        S = N // tau + (1 if N % tau else 0)
        for j in range(S):
            rows.append([members[((j * tau + k) * N) // (S * tau)] for k in range(tau)])
    return np.array(rows, dtype=np.int32)


@pytest.mark.parametrize("grid,window,batch,n,tau", [
    ((20, 17, 1), (6, 5, 1), 1, 200, 7),
    ((9, 9, 6), (4, 4, 3), 2, 500, 10),
    ((64, 64, 1), (12, 12, 1), 1, 2000, 36),
    ((5, 5, 5), (5, 5, 5), 1, 125, 36),
])
def test_partition_vs_brute_force(oracle, grid, window, batch, n, tau):
    rng = np.random.default_rng(7)
    coords = di.unique_cells(rng, n, grid, batch)
    for axis in (0, 1):
        p = oracle.partition(coords, batch, grid, window, tau, axis)
        want = _brute_partition(coords, batch, grid, window, tau, axis)
        assert np.array_equal(p.set_table, want)
        # bookkeeping arrays
        assert p.win_count.sum() == n and p.win_start[-1] == n and p.win_setoff[-1] == p.num_sets
        assert np.array_equal(np.diff(p.win_start), p.win_count)
        assert np.array_equal(np.diff(p.win_setoff), -(-p.win_count // tau))
        assert np.array_equal(np.sort(p.perm), np.arange(n))


def test_partition_invariants(oracle):
    """Every voxel lands in exactly one set; sets of a window cover exactly its voxels; the two
    rotated partitions differ only in the sort axis (same windows, same N, same S, same members)."""
    cfg = di.make_config(1)
    coords, grid, window, tau = cfg["coords"], cfg["grid"], cfg["window"], cfg["set_size"]
    n = coords.shape[0]
    p0 = oracle.partition(coords, 1, grid, window, tau, 0)
    p1 = oracle.partition(coords, 1, grid, window, tau, 1)
    assert np.array_equal(p0.win_count, p1.win_count)
    assert np.array_equal(p0.win_setoff, p1.win_setoff)
    wid = (coords[:, 1] // window[0]) * 6 + coords[:, 2] // window[1]
    for p in (p0, p1):
        seen = np.zeros(n, dtype=np.int64)
        for row in p.set_table:
            u = np.unique(row)
            seen[u] += 1
            assert len(set(wid[u].tolist())) == 1  # window-bounded
        assert np.all(seen == 1)
        assert p.num_sets <= n // tau + np.count_nonzero(p.win_count)
    for w in range(36):
        s0, s1 = p0.win_setoff[w], p0.win_setoff[w + 1]
        m0 = np.unique(p0.set_table[s0:s1])
        m1 = np.unique(p1.set_table[s0:s1])
        assert np.array_equal(m0, m1)
        assert np.array_equal(m0, np.flatnonzero(wid == w))
    # the axis-1 order of (x, y) equals the axis-0 order of the transposed frame
    swapped = coords.copy()
    swapped[:, 1], swapped[:, 2] = coords[:, 2], coords[:, 1]
    pt = oracle.partition(swapped, 1, (grid[1], grid[0], grid[2]), (window[1], window[0], window[2]), tau, 0)
    for w in range(36):
        wx, wy = divmod(w, 6)
        wt = wy * 6 + wx
        a = p1.set_table[p1.win_setoff[w]:p1.win_setoff[w + 1]]
        b = pt.set_table[pt.win_setoff[wt]:pt.win_setoff[wt + 1]]
        assert np.array_equal(a, b)


def test_partition_permutation_equivariance(oracle):
    rng = np.random.default_rng(3)
    coords = di.unique_cells(rng, 300, (30, 30, 2), 1)
    sh = rng.permutation(300)
    p = oracle.partition(coords, 1, (30, 30, 2), (7, 7, 2), 5, 0)
    ps = oracle.partition(coords[sh], 1, (30, 30, 2), (7, 7, 2), 5, 0)
    assert np.array_equal(sh[ps.set_table], p.set_table)


def test_partition_errors(oracle):
    bad = np.array([[0, 9, 0, 0]], dtype=np.int32)
    with pytest.raises(ValueError):
        oracle.partition(bad, 1, (8, 8, 1), (4, 4, 1), 3, 0)
    ok = np.array([[0, 1, 1, 0], [0, 2, 2, 0], [0, 7, 7, 0]], dtype=np.int32)
    with pytest.raises(ValueError):
        oracle.partition(ok, 1, (8, 8, 1), (4, 4, 1), 1, 0, cap_sets=2)
    empty = oracle.partition(np.zeros((0, 4), dtype=np.int32), 1, (8, 8, 1), (4, 4, 1), 3, 0)
    assert empty.num_sets == 0 and empty.win_count.sum() == 0
