"""The N > 1 path of bench.py is replicas only: no data-path collective, just max-over-ranks timing and summed
units.  Checked here with two gloo ranks on CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms, e2e, launches = bench.aggregate_over_ranks(10.0 + 5.0 * rank, 0.02 + 0.01 * rank, 100 + rank, world, "cpu")
        dist.barrier()
        out.put((rank, ms, e2e, launches, bench.whole_job_rate(world, 32 * 20, ms / 1e3)))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_take_the_slowest_time_and_sum_the_units():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, e2e, launches, rate in res:
        assert ms == 15.0 and abs(e2e - 0.03) < 1e-12 and launches == 201
        assert abs(rate - 2 * 640 / 0.015) < 1e-6


def test_single_rank_is_untouched():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate_over_ranks(3.0, 0.5, 7, 1, "cpu") == (3.0, 0.5, 7)
    assert bench.whole_job_rate(1, 640, 0.004) == 160000.0
