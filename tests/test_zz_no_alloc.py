"""dsvt_partition_noalloc against dsvt_partition (and the CPU oracle), through the C ABI.

The no-allocation entry point serves callers that are not allowed to allocate device memory (fixed
memory budgets, foreign allocators, plug-ins given only a stream and buffers).  Its workspace is one
fixed array inside the library that every call shares and that keeps the last call's contents, so the
check runs two different calls back to back: the second must not see anything of the first.
Collected last on purpose (file name), so a failure here cannot hide another test's result.
"""
import numpy as np
import pytest
import torch

import dsvt_inputs as di

pytestmark = pytest.mark.gpu


def _blank_table(api, cap, tau):
    return api.SetTable(torch.full((cap, tau), -1, dtype=torch.int32, device="cuda"),
                        torch.full((1,), -1, dtype=torch.int32, device="cuda"),
                        torch.full((4 * cap + 4,), -1, dtype=torch.int32, device="cuda"), cap, tau)


def _same(api, ctx, coords, batch, grid, window, tau, axis, check_memory=True, oracle=None):
    dc = torch.from_numpy(coords).cuda()
    n = coords.shape[0]
    want = ctx.partition(dc, batch, grid, window, tau, axis, out=_blank_table(api, max(n, 1), tau))
    assert ctx.status_sync() == 0
    got = _blank_table(api, max(n, 1), tau)
    bits = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    free_before = torch.cuda.mem_get_info()[0]
    api.partition_noalloc(dc, batch, grid, window, tau, axis, got, status_bits=bits)
    torch.cuda.synchronize()
    if check_memory:  # (the very first call on a device may make the driver load the library's image)
        took_none = torch.cuda.mem_get_info()[0] == free_before
        if not took_none:  # free memory is device-wide: something else may have moved it; look once more
            free_before = torch.cuda.mem_get_info()[0]
            api.partition_noalloc(dc, batch, grid, window, tau, axis, got, status_bits=bits)
            torch.cuda.synchronize()
            took_none = torch.cuda.mem_get_info()[0] == free_before
        assert took_none  # the call took no device memory
    assert int(bits.item()) == 0
    S = int(want.num_sets.item())
    assert int(got.num_sets.item()) == S
    assert torch.equal(got.set_table[:S], want.set_table[:S])  # integer outputs: bit-exact
    assert torch.equal(got.set_rowoff[: S + 1], want.set_rowoff[: S + 1])
    cap = want.cap_sets  # the tile plan behind the row offsets: tile count, tile starts, terminator
    head = int(want.set_rowoff[cap + 1].item())
    tiles = head & ~0x40000000 if head >= 0 else 0
    assert torch.equal(got.set_rowoff[cap + 1: cap + 3 + tiles], want.set_rowoff[cap + 1: cap + 3 + tiles])
    if head >= 0 and head & 0x40000000:  # a plan over reordered sets: the order and the rows before each position
        assert torch.equal(got.set_rowoff[2 * cap + 3: 2 * cap + 3 + S], want.set_rowoff[2 * cap + 3: 2 * cap + 3 + S])
        assert torch.equal(got.set_rowoff[3 * cap + 3: 3 * cap + 4 + S], want.set_rowoff[3 * cap + 3: 3 * cap + 4 + S])
    assert torch.all(got.set_table[S:] == -1)  # nothing written past the last set
    if oracle is not None:  # and against the CPU oracle directly, not only through dsvt_partition
        ref = oracle.partition(coords, batch, grid, window, tau, axis)
        assert S == ref.set_table.shape[0]
        assert np.array_equal(got.set_table[:S].cpu().numpy(), ref.set_table)
    return S


def test_no_alloc_partition_matches_partition_on_two_calls_in_a_row(oracle):
    from paper_2301_06051_b200 import api

    assert torch.cuda.is_available()
    api.load()
    big = di.make_config(2)  # 32,000 pillars, 1521 windows
    small = di.make_config(1)  # 2,000 pillars, 36 windows: far fewer windows and voxels than the call before
    ctx = api.Context(big["n"], 2048, 64)
    _same(api, ctx, small["coords"], 1, small["grid"], small["window"], 36, 0, check_memory=False)
    s_big = _same(api, ctx, big["coords"], 1, big["grid"], big["window"], 36, 0, oracle=oracle)
    s_small = _same(api, ctx, small["coords"], 1, small["grid"], small["window"], 36, 1, oracle=oracle)
    assert s_big > s_small > 0
    _same(api, ctx, big["coords"], 1, big["grid"], big["window"], 36, 1)
    # an empty frame right after a full one
    _same(api, ctx, np.zeros((0, 4), dtype=np.int32), 1, (8, 8, 1), (4, 4, 1), 3, 0)


def test_no_alloc_partition_rejects_sizes_beyond_its_fixed_workspace():
    from paper_2301_06051_b200 import api

    api.load()
    too_many = torch.zeros((api.NOALLOC_MAX_VOXELS + 1, 4), dtype=torch.int32, device="cuda")
    out = _blank_table(api, 8, 36)
    with pytest.raises(api.DsvtError) as e:
        api.partition_noalloc(too_many, 1, (468, 468, 1), (12, 12, 1), 36, 0, out)
    assert e.value.code == -2
    few = torch.zeros((4, 4), dtype=torch.int32, device="cuda")
    with pytest.raises(api.DsvtError) as e:
        api.partition_noalloc(few, 1, (4096, 4096, 1), (2, 2, 1), 36, 0, out)  # 4M windows
    assert e.value.code == -2
    # a bad coordinate is reported through the caller's status word, as with dsvt_partition
    bad = torch.tensor([[0, 1, 1, 0], [0, 99, 1, 0]], dtype=torch.int32, device="cuda")
    bits = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.partition_noalloc(bad, 1, (8, 8, 1), (4, 4, 1), 3, 0, out, status_bits=bits)
    assert int(bits.item()) & api.STATUS_BAD_COORD
    ok = torch.tensor([[0, 1, 1, 0], [0, 2, 1, 0]], dtype=torch.int32, device="cuda")
    api.partition_noalloc(ok, 1, (8, 8, 1), (4, 4, 1), 3, 0, out, status_bits=bits)
    assert int(bits.item()) == 0  # the status of the previous call does not leak into this one
