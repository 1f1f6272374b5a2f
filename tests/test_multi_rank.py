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


def test_gpus_flag_starts_one_replica_per_gpu(tmp_path):
    """`bench.py --gpus N` started as a plain process re-launches itself as N ranks of one
    node.  The same launcher runs a stand-in script here (gloo, CPU): two processes come up with
    RANK / WORLD_SIZE set, meet in the barrier, and the job's time is the slower replica's."""
    sys.path.insert(0, ROOT)
    import json
    import bench
    out = tmp_path / "out.json"
    cmd = bench.replica_command(2, os.path.join(ROOT, "tests", "replica_stub.py"), [str(out), "--steps", "3"], 29400)
    assert cmd[1:4] == ["-m", "torch.distributed.run", "--nnodes=1"] and "127.0.0.1" in cmd
    rc = bench.spawn_replicas(2, os.path.join(ROOT, "tests", "replica_stub.py"), [str(out), "--steps", "3"],
                              port=29400 + os.getpid() % 500)
    assert rc == 0
    res = json.loads(out.read_text())
    assert res["world"] == 2 and res["ms"] == 3.0 and res["value"] == 2 * 100 / 3e-3
    assert res["args"] == ["--steps", "3"]
