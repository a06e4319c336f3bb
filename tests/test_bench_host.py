"""Host-side logic of the multi-GPU bench path, on CPU: two gloo ranks (the path shards by frame, so
the only cross-rank step is the max over ranks of the step time)."""
import io
import os
import sys
from contextlib import redirect_stdout

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench

    mine = [10.0 + 5.0 * rank, 3.0 - rank]  # rank 1 is slower on the first, faster on the second
    got = bench.max_over_ranks(mine)
    out.put((rank, got, bench.job_throughput(world, 1000, got[0])))
    dist.barrier()
    dist.destroy_process_group()


def test_step_time_is_the_max_over_ranks_and_value_is_the_whole_job():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29000 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, got, value in res:
        assert got == [15.0, 3.0]
        assert abs(value - 2 * 1000 / 15e-3) < 1e-6  # both ranks' units over the slowest rank's time


def test_single_process_needs_no_process_group():
    import bench

    assert bench.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert bench.job_throughput(1, 32000 * 4, 2.0) == 32000 * 4 / 2e-3


def test_reference_arm_runs_on_rank_zero_only(monkeypatch):
    import bench

    monkeypatch.setenv("RANK", "1")
    monkeypatch.setenv("WORLD_SIZE", "2")
    buf = io.StringIO()
    with redirect_stdout(buf):
        bench.run_reference(type("A", (), {"config": 1, "steps": 1, "warmup": 0, "gpus": 2})())
    assert buf.getvalue() == ""  # other ranks exit without work


def test_algorithmic_flops_formula():
    import numpy as np

    import bench

    # two sets of 3 and 5 distinct voxels, C = 8, hidden = 16: 8 voxels * (8*64 + 4*8*16) + 4*8*(9 + 25)
    assert bench.algorithmic_flops_per_layer(np.array([0, 3, 8]), 8, 16) == 8 * (512 + 512) + 32 * 34
