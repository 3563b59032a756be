"""The N > 1 path of the bench on CPU: two gloo ranks stand in for two GPUs.  The hot path shards as
independent replicas (no data-path collective); what the ranks share is the timing rule: the job takes as
long as its slowest rank and does the sum of the ranks' work."""
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
    # rank 1 is the slow one: 10 sweeps in 30 ms against 20 ms on rank 0
    total_ms, e2e_ms = (20.0, 100.0) if rank == 0 else (30.0, 80.0)
    ms_per_step, value, e2e = bench.aggregate_replicas(total_ms, e2e_ms, 10, dist, "cpu")
    dist.barrier()
    dist.destroy_process_group()
    out[rank] = (ms_per_step, value, e2e)


def test_replica_aggregation_takes_slowest_rank_and_sums_work():
    world, port = 2, 29500 + os.getpid() % 2000
    with mp.get_context("spawn").Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = [out[r] for r in range(world)]
    assert res[0] == res[1]                                  # every rank holds the job's numbers
    ms_per_step, value, e2e = res[0]
    assert abs(ms_per_step - 3.0) < 1e-12                    # slowest rank: 30 ms / 10 sweeps
    assert abs(value - 2 / 3.0e-3) < 1e-6                    # two image pairs per 3 ms
    assert abs(e2e - 2 / 100.0e-3) < 1e-6                    # slowest end-to-end time (rank 0's)


def test_single_process_aggregation_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    ms_per_step, value, e2e = bench.aggregate_replicas(50.0, 200.0, 10)
    assert ms_per_step == 5.0 and abs(value - 200.0) < 1e-9 and abs(e2e - 5.0) < 1e-9
