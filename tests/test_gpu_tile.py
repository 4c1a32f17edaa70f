"""GPU parity of the tcgen05 / TMEM tile path (W4A16_PATH_TILE) against the FP64 oracle (Eq. 2;
Algorithm 1 Split-K), through the C ABI: every batch-tile width, ragged batch and column tails,
whole-K and Split-K, and the prefill configuration at full size on sampled columns."""
import numpy as np
import pytest
import torch

import oracle
from paper_2601_16536_b200 import binding as B
from paper_2601_16536_b200 import workloads as wl
from gpu_util import assert_close, c_bits, c_f64, ensure_ws, pack_problem, to_dev

pytestmark = pytest.mark.gpu


def _run(d, M, N, K, split_k, path=B.PATH_TILE):
    pw = pack_problem(d, N, K)
    ws = ensure_ws(M, N, K, split_k)
    C = B.w4a16_gemm(to_dev(d["A"]), pw, split_k=split_k, path=path)
    torch.cuda.synchronize()
    assert B.w4a16_device_status() == 0
    del ws
    return C


# (M, K, N): batch tiles of 16 / 32 / 64 / 128 / 256 rows with ragged tails, one and several column
# tiles, a 64-column tail tile (N = 192, 320), one to many groups
SHAPES = [(32, 128, 128), (1, 256, 128), (9, 640, 192), (16, 1152, 256), (17, 640, 192), (33, 384, 256), (64, 1152, 128),
          (100, 896, 320), (128, 512, 256), (129, 768, 128), (256, 2048, 384), (300, 1280, 192),
          (700, 640, 256),
          # wide enough (twelve column tiles and more) for the 128- and 256-row batch tiles themselves
          (120, 512, 1536), (300, 384, 1600),
          # wide enough for 64-row batch tiles (more than 24 column tiles), with a 64-column tail tile
          (64, 640, 3328), (40, 1152, 3392)]


@pytest.mark.parametrize("M,K,N", SHAPES)
@pytest.mark.parametrize("split_k", [1, 0, 2, 3])
def test_tile_path_matches_oracle(M, K, N, split_k):
    if split_k > K // 128:
        pytest.skip("more splits than groups")
    d = wl.make_problem(M, K, N, seed=7000 + M + K + N)
    C = _run(d, M, N, K, split_k)
    ref = oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, 128)
    assert_close(c_f64(C), ref, "tile M%d K%d N%d S%d" % (M, K, N, split_k))


@pytest.mark.parametrize("split_k", [2, 0, 1])
def test_tile_path_many_chunks_per_cta(split_k):
    # more tiles than SMs.  Classic split: every CTA walks several chunks through the same rings.
    # Balanced: a chunk is about 2.2 units of a 2-unit tile, so chunks hold whole tiles and partial
    # segments of both neighbours.
    M, K, N = 40, 256, 128 * 160
    d = wl.make_problem(M, K, N, seed=7100)
    C = _run(d, M, N, K, split_k)
    ref = oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, 128)
    assert_close(c_f64(C), ref, "tile many chunks, split_k=%d" % split_k)


def test_tile_path_exact_inputs_bit_equal_for_every_split():
    M, K, N = 70, 2304, 256
    d = wl.make_exact_problem(M, K, N, seed=7200)
    want = oracle.gemm_int(d["A_int"], d["Wq"], d["E"], d["Z"], M, N, K, 128)
    for split_k in (1, 0, 2, 4, 5, 9, 18):
        C = _run(d, M, N, K, split_k)
        assert np.array_equal(c_bits(C), want), "split_k=%d" % split_k


def test_wide_batch_tiles_with_slices_bit_equal_for_every_split():
    # Twelve column tiles keep the 256-row batch tile, and its K slices are summed by the second kernel
    # (tile_splitk_reduce_kernel) instead of inside the GEMM kernel: same order, so with exact inputs the same
    # bits as one slice, for a ragged batch (200 of 256 rows) and a ragged slice count (8 groups in 3 slices).
    M, K, N = 200, 1024, 1536
    d = wl.make_exact_problem(M, K, N, seed=7250)
    want = oracle.gemm_int(d["A_int"], d["Wq"], d["E"], d["Z"], M, N, K, 128)
    for split_k in (1, 0, 2, 3, 4, 8):
        C = _run(d, M, N, K, split_k)
        assert np.array_equal(c_bits(C), want), "split_k=%d" % split_k


def test_tile_path_bit_identical_run_to_run():
    M, K, N = 96, 4096, 512
    d = wl.make_problem(M, K, N, seed=7300)
    pw = pack_problem(d, N, K)
    A = to_dev(d["A"])
    ws = ensure_ws(M, N, K, (0, 1, 8))
    for split_k in (0, 1, 8):
        first = c_bits(B.w4a16_gemm(A, pw, split_k=split_k, path=B.PATH_TILE))
        for _ in range(4):
            assert np.array_equal(first, c_bits(B.w4a16_gemm(A, pw, split_k=split_k, path=B.PATH_TILE)))
    del ws


@pytest.mark.parametrize("M", [256, 1024, 4096])
def test_prefill_config_full_size_sampled_columns(M):
    # config 5 (K = N = 8192) in the launch configuration the benchmark times (automatic path and
    # split); the oracle computes whole columns of C, sampled at tile edges and interiors
    case = [c for c in wl.cases_of(5) if c.M == M][0]
    d = wl.make_case(case)
    K, N = case.K, case.N
    pw = pack_problem(d, N, K)
    ws = ensure_ws(M, N, K, 0)
    C = B.w4a16_gemm(to_dev(d["A"]), pw)
    torch.cuda.synchronize()
    assert B.w4a16_device_status() == 0
    got = c_f64(C)
    per = 2 if M >= 4096 else 4
    for n0 in (0, 126, 4095, N - per):
        ref = oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, 128, cols=(n0, n0 + per))
        assert_close(got[:, n0:n0 + per], ref[:, n0:n0 + per], "prefill M%d cols %d" % (M, n0))
    del ws
