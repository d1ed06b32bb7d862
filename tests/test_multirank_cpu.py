"""The multi-rank part of bench.py (replicas only: no data-path collective, one MAX reduction of the timing) on two
gloo ranks on the CPU."""
import os
import sys

import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    local_ms = 100.0 if rank == 0 else 250.0           # rank 1 is the slow replica
    qps, ms = bench.whole_job_qps(local_ms, 512, dist)
    out[rank] = (qps, ms)
    dist.barrier()
    dist.destroy_process_group()


def test_whole_job_qps_is_all_queries_over_the_slowest_rank():
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_rank, args=(world, 29531 + os.getpid() % 200, out), nprocs=world, join=True)
        for r in range(world):
            qps, ms = out[r]
            assert ms == 250.0 and abs(qps - 2 * 512 / 0.25) < 1e-6


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    qps, ms = bench.whole_job_qps(50.0, 256)
    assert ms == 50.0 and abs(qps - 5120.0) < 1e-9
