"""The benchmark's cross-rank logic on CPU: two gloo ranks, each a replica with its own timing.
The path has no data-path collective (units are independent); ranks only agree on the slowest time."""
import os
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = 10.0 + 5.0 * rank                     # rank 1 is slower
    slowest = bench.max_over_ranks(mine, "cpu")
    out[rank] = (slowest, bench.whole_job_gbs(1e9, slowest * 1e-3, world))
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_and_weak_scaling_value():
    world, port = 2, 29731
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == res[1][0] == 15.0                      # both ranks see the slowest replica's time
    assert abs(res[0][1] - 2 * 1e9 / 15e-3 / 1e9) < 1e-9       # whole-job throughput = ranks x per-rank bytes / time


def test_single_process_passthrough():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.whole_job_gbs(2e9, 1e-3, 1) == 2000.0
