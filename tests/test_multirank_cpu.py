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


def test_bench_gpus_n_starts_n_ranks_itself():
    """`bench.py --gpus N` outside a launcher starts N ranks (one process per GPU).  --dry-launch runs the same launch
    and the same timing reduction with gloo ranks on the CPU: rank r reports 100 + 50 r ms for 512 queries."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_PORT")}
    for n in (2, 3):
        r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", str(n), "--dry-launch"],
                           capture_output=True, text=True, env=env, timeout=300)
        assert r.returncode == 0, r.stderr[-2000:]
        lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
        assert len(lines) == 1                                   # rank 0 alone prints
        d = json.loads(lines[0])
        slowest = 100.0 + 50.0 * (n - 1)
        assert d["n_gpus"] == n and d["ms"] == slowest and abs(d["value"] - n * 512 / (slowest / 1e3)) < 1e-6
