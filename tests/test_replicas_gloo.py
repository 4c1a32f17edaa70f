"""The N > 1 path of bench.py on CPU: the GEMM has no exchange step, so ranks are independent
replicas and the only cross-rank logic is "time = slowest rank, value = all ranks' bytes / that
time".  Two gloo ranks on 127.0.0.1 exercise exactly that code."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert bench._rank_world()[:2] == (rank, world)
        mine = 0.010 * (rank + 1)                     # rank 1 is the slow one
        dist.barrier()
        slowest = bench.max_over_ranks(mine, dist, "cpu")
        value = bench.whole_job_value(1_000_000_000, 10, world, slowest)
        with open(os.path.join(out_dir, "r%d.txt" % rank), "w") as f:
            f.write("%.9f %.6f" % (slowest, value))
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank_and_the_aggregate(tmp_path):
    world, port = 2, 29611 + os.getpid() % 200
    mp.spawn(_rank_main, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    for r in range(world):
        slowest, value = (float(x) for x in open(tmp_path / ("r%d.txt" % r)).read().split())
        assert abs(slowest - 0.020) < 1e-9                      # max over ranks, on every rank
        assert abs(value - 1e9 * 10 * 2 / 0.020 / 1e9) < 1e-3   # both ranks' bytes over that time


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(0.5, None, "cpu") == 0.5
    assert bench.whole_job_value(2e9, 3, 1, 0.5) == 12.0
