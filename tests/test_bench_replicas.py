"""Host logic of the multi-replica benchmark path (N > 1: independent replicas, no exchange step):
the slowest rank's time is what every rank reports, and the aggregate counts every replica.
Runs two gloo ranks on the CPU."""
import os
import sys

import pytest
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    mine = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    got = bench.max_over_ranks(mine, world)
    dist.barrier()
    out.put((rank, mine, got))
    dist.destroy_process_group()


def test_max_over_ranks_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [10.0, 15.0]
    assert [r[2] for r in res] == [15.0, 15.0]    # both ranks report the slowest time


def test_whole_job_value_counts_every_replica():
    sys.path.insert(0, ROOT)
    import bench
    one = bench.whole_job_tops(1, 4096, 4096, 4096, 1.25)
    assert one == pytest.approx(2 * 4096 ** 3 / 1.25e-3 / 1e12)
    assert bench.whole_job_tops(8, 4096, 4096, 4096, 1.25) == pytest.approx(8 * one)
    assert bench.max_over_ranks(3.5, 1) == 3.5    # single rank: no process group needed
