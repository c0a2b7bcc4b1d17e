"""The only cross-rank step of the benchmark (max of the times, sum of the tokens) on two gloo
ranks on CPU.  The verify step itself does not shard: every rank runs an independent replica."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms, tokens = bench.reduce_over_ranks(10.0 + 5.0 * rank, 100.0 + rank, "cpu")
    out[rank] = (ms, tokens)
    dist.destroy_process_group()


def test_two_ranks_take_max_time_and_sum_tokens():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, 29611, out), nprocs=world, join=True)
    assert out[0] == out[1] == (15.0, 201.0)


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_over_ranks(3.5, 7.0, "cpu") == (3.5, 7.0)
