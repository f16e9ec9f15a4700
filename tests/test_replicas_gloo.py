"""The benchmark's multi-rank path on CPU: two gloo ranks, each an independent replica (the hot
path has no exchange step), timings reduced with a maximum over ranks, value = the sum of what
all ranks processed divided by that time."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        local = [10.0 + rank, 3.0 - rank, 7.0]             # rank-dependent timings (ms)
        got = bench.max_over_ranks(local, "cpu")
        value = bench.aggregate_value(world, K=8, d=1000, t_step_ms=got[0])
        out.put((rank, got, value))
    finally:
        dist.destroy_process_group()


@pytest.mark.timeout(120)
def test_two_replicas_take_the_slowest_time_and_sum_the_work():
    world, port = 2, 29731 + os.getpid() % 1000
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=100) for _ in range(world))
    for p in procs:
        p.join(30)
        assert p.exitcode == 0
    for rank, got, value in results:
        assert got == [11.0, 3.0, 7.0]                      # element-wise max over the two ranks
        # 2 ranks x (8 + 1) x 4 x 1000 bytes in 11 ms
        assert value == pytest.approx(2 * 9 * 4000 / 11e-3 / 1e9)


def test_single_process_needs_no_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5], "cpu") == [1.5, 2.5]
    assert bench.aggregate_value(1, 8, 25_557_032, 1.0) == pytest.approx(9 * 4 * 25_557_032 / 1e-3 / 1e9)
