"""The benchmark's multi-rank bookkeeping on CPU: two gloo ranks, MAX over ranks, replicas-only aggregate."""
import os
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.reduce_over_ranks(10.0 + 5.0 * rank, dist, "cpu")      # rank 1 is the slow one
    dist.barrier()
    out[rank] = (ms, bench.whole_job_value(256, world, ms))
    dist.destroy_process_group()


def test_two_ranks_take_the_slowest_time_and_add_their_tokens():
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_rank, args=(world, 29500 + os.getpid() % 2000, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == res[1][0] == 15.0                             # both ranks agree on the MAX
    assert abs(res[0][1] - 2 * 256 / 15e-3) < 1e-6                   # two replicas' tokens over the slowest rank's time


def test_single_rank_passthrough():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_over_ranks(3.5) == 3.5
    assert bench.whole_job_value(100, 1, 50.0) == 2000.0
