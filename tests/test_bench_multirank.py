"""The N > 1 path of bench.py is replicas only (no data-path collective): what ranks share is the timing rule
(max over ranks) and the whole-job rate.  Checked here with two gloo ranks on CPU."""
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
    ms = bench.max_over_ranks(1.0 + rank, dist, "cpu")            # rank 1 is the slow one
    rate = bench.whole_job_rate(1000, world, ms)
    dist.barrier()
    dist.destroy_process_group()
    out[rank] = (ms, rate)


def test_slowest_rank_sets_the_time_and_rate_is_the_aggregate():
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, 29533, out), nprocs=world, join=True)
        assert out[0] == out[1]
        ms, rate = out[0]
        assert ms == 2.0
        assert abs(rate - 2 * 1000 / 2e-3) < 1e-6


def test_single_rank_is_a_no_op():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, None, "cpu") == 3.5
    assert bench.whole_job_rate(16384, 1, 0.5) == 16384 / 0.5e-3
