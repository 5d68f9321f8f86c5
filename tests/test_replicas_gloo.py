"""The multi-GPU mode of the benchmark is "replicas only": every rank runs the whole path on its own data and
the only communication is the max-over-ranks of the measured time.  This checks that host logic with two
gloo ranks on CPU: the slowest rank's time is what every rank sees, and the aggregate counts every replica."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = 0.010 * (rank + 1)                      # rank 1 is twice as slow
    t = bench.max_over_ranks(mine, dist, torch.device("cpu"))
    out[rank] = (t, bench.whole_job_gbs(world, 25_000_000, t, 10))
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_and_aggregate_with_two_gloo_ranks():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, 29611 + os.getpid() % 200, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for rank in (0, 1):
        t, gbs = res[rank]
        assert abs(t - 0.020) < 1e-12                              # the slower rank's time, on both ranks
        assert abs(gbs - 2 * 25_000_000 / (0.020 / 10) * 1e-9) < 1e-9


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(0.5, None, None) == 0.5
    assert bench.whole_job_gbs(1, 10**9, 1.0, 1) == 1.0
