"""Host-side logic of the multi-GPU benchmark path, on CPU with gloo (world size 2).

The path has no exchange step: ranks run independent replicas.  What is shared is
the timing rule (barrier, then the maximum of the per-rank times) and the whole-job
throughput computed from it."""
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
    dist.barrier()
    ms = bench.max_over_ranks(3.0 + 2.0 * rank)     # rank 1 is the slow replica
    out[rank] = (ms, bench.aggregate_tokens_per_s(8192, world, ms))
    dist.destroy_process_group()


def test_timing_is_max_over_ranks_and_throughput_aggregates():
    world = 2
    port = 29500 + os.getpid() % 2000
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == res[1][0] == 5.0
    assert res[0][1] == res[1][1] == 2 * 8192 / 5e-3


def test_single_process_is_a_no_op():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(1.25) == 1.25
    assert bench.aggregate_tokens_per_s(8192, 1, 2.0) == 8192 / 2e-3
