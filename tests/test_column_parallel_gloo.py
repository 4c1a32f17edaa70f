"""N-sharded (column-parallel) multi-GPU use of the GEMM, checked on CPU with two gloo ranks: the shard
arithmetic, the slicing of the raw arrays and the all-gather that assembles C.  Each rank's slice of C is
produced here by the oracle on the rank's own weight columns (the CUDA call it stands in for computes the
same columns); the assembled result must equal the oracle's whole product."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_shards_are_whole_tiles_and_cover_every_column_once():
    sys.path.insert(0, ROOT)
    from paper_2601_16536_b200 import parallel as par
    for N in (64, 1536, 4096, 22016, 12288):
        for world in (1, 2, 3, 4, 8):
            if N // 64 < world:
                continue
            s = par.column_shards(N, world)
            assert s[0][0] == 0 and s[-1][1] == N
            assert all(a % 64 == 0 and b % 64 == 0 and b > a for a, b in s)
            assert all(s[i][1] == s[i + 1][0] for i in range(world - 1))
            widths = [b - a for a, b in s]
            assert max(widths) - min(widths) <= 64


def _rank_main(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    import oracle
    from paper_2601_16536_b200 import parallel as par
    from paper_2601_16536_b200 import workloads as wl
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        M, K, N = 3, 256, 192            # three tiles over two ranks: shards of 128 and 64 columns
        d = wl.make_problem(M, K, N, seed=5)
        n0, n1 = par.column_shard(N, world, rank)
        wq, s, z = par.shard_raw_weights(d["Wq"], d["S"], d["Z"], n0, n1)
        local = oracle.gemm(d["A"], np.ascontiguousarray(wq), np.ascontiguousarray(s), np.ascontiguousarray(z),
                            M, n1 - n0, K, 128)
        whole = par.gather_columns(torch.from_numpy(local), N, dist, world, rank).numpy()
        np.save(os.path.join(out_dir, "r%d.npy" % rank), whole)
    finally:
        dist.destroy_process_group()


def test_two_ranks_assemble_the_whole_product(tmp_path):
    world, port = 2, 29811 + os.getpid() % 150
    mp.spawn(_rank_main, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    sys.path.insert(0, ROOT)
    import oracle
    from paper_2601_16536_b200 import workloads as wl
    d = wl.make_problem(3, 256, 192, seed=5)
    want = oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], 3, 192, 256, 128)
    for r in range(world):
        assert np.array_equal(np.load(tmp_path / ("r%d.npy" % r)), want)
