"""GPU parity of w4a16_gemm against the FP64 oracle (Eq. 2; Algorithm 1 Split-K), through the C ABI.

Tolerances: relative Frobenius error <= 1e-3 and per element |dC| <= 2e-3 (1 + |C_ref|) against the
FP64-accumulated oracle.  With exactly representable inputs the result is unique and must be
bit-equal for every path and split.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2601_16536_b200 import binding as B
from paper_2601_16536_b200 import workloads as wl
from gpu_util import assert_close, c_bits, c_f64, ensure_ws, pack_problem, to_dev

pytestmark = pytest.mark.gpu

PATHS = {"simple": B.PATH_SIMPLE, "decode": B.PATH_DECODE}


def _run(d, M, N, K, split_k, path):
    pw = pack_problem(d, N, K)
    ws = ensure_ws(M, N, K, split_k)
    C = B.w4a16_gemm(to_dev(d["A"]), pw, split_k=split_k, path=path)
    torch.cuda.synchronize()
    assert B.w4a16_device_status() == 0
    del ws
    return C


# several 64-column tiles, ragged group counts (5, 7, 9 groups: not a multiple of the 4 groups a
# stage holds, nor of the splits), every batch-block edge
SMALL = [(1, 128, 64), (1, 640, 192), (3, 896, 128), (8, 1152, 256), (9, 640, 128),
         (16, 1152, 192), (5, 4096, 512)]


@pytest.mark.parametrize("path", list(PATHS))
@pytest.mark.parametrize("M,K,N", SMALL)
@pytest.mark.parametrize("split_k", [0, 1, 2, 3])
def test_small_shapes_match_oracle(path, M, K, N, split_k):
    if split_k > K // 128:
        pytest.skip("more splits than groups")
    d = wl.make_problem(M, K, N, seed=M * 1000 + K + N)
    C = _run(d, M, N, K, split_k, PATHS[path])
    ref = oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, 128)
    assert_close(c_f64(C), ref, "%s M%d K%d N%d S%d" % (path, M, K, N, split_k))


@pytest.mark.parametrize("path", list(PATHS))
@pytest.mark.parametrize("M", [17, 33, 64])
def test_batch_larger_than_one_block(path, M):
    K, N = 768, 128
    d = wl.make_problem(M, K, N, seed=M)
    C = _run(d, M, N, K, 2, PATHS[path])
    ref = oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, 128)
    assert_close(c_f64(C), ref, "%s M%d" % (path, M))


@pytest.mark.parametrize("path", list(PATHS))
def test_exact_inputs_are_bit_equal_for_every_split(path):
    # A in {-1,0,1}, s = 2^e: every partial sum is exact in FP32 in any order, so the FP16
    # result is unique (closed form) -- any split, any path must return exactly it
    M, K, N = 7, 2304, 192    # 18 groups
    d = wl.make_exact_problem(M, K, N, seed=90)
    want = oracle.gemm_int(d["A_int"], d["Wq"], d["E"], d["Z"], M, N, K, 128)
    for split_k in (0, 1, 2, 4, 5, 8, 16, 18):
        C = _run(d, M, N, K, split_k, PATHS[path])
        assert np.array_equal(c_bits(C), want), "split_k=%d" % split_k


@pytest.mark.parametrize("path", list(PATHS))
def test_q_equals_z_gives_zero_and_scaling_is_linear(path):
    M, K, N = 4, 512, 128
    d = wl.make_problem(M, K, N, seed=91)
    dz = dict(d)
    dz["Wq"] = np.repeat(d["Z"].astype(np.uint32) * np.uint32(0x11111111), 16, axis=0)
    C0 = _run(dz, M, N, K, 1, PATHS[path])
    assert np.all(c_f64(C0) == 0.0)
    d2 = dict(d)
    d2["S"] = (d["S"].view(np.float16) * np.float16(2)).view(np.uint16)
    C1 = c_f64(_run(d, M, N, K, 1, PATHS[path]))
    C2 = c_f64(_run(d2, M, N, K, 1, PATHS[path]))
    assert np.array_equal(C2, 2.0 * C1)   # power-of-two scaling commutes with every rounding


def test_results_are_bit_identical_run_to_run():
    M, K, N = 16, 11008, 512
    d = wl.make_problem(M, K, N, seed=92)
    pw = pack_problem(d, N, K)
    A = to_dev(d["A"])
    ws = ensure_ws(M, N, K, (0, 16))
    for split_k in (0, 1, 4, 16):
        first = c_bits(B.w4a16_gemm(A, pw, split_k=split_k, path=B.PATH_DECODE))
        for _ in range(5):
            again = c_bits(B.w4a16_gemm(A, pw, split_k=split_k, path=B.PATH_DECODE))
            assert np.array_equal(first, again)
    del ws


def test_auto_path_and_split_match_oracle():
    for M, K, N in [(1, 4096, 4096), (4, 11008, 1024), (16, 2048, 2048)]:
        d = wl.make_problem(M, K, N, seed=93 + M)
        C = _run(d, M, N, K, 0, B.PATH_AUTO)
        ref = oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, 128)
        assert_close(c_f64(C), ref, "auto M%d K%d N%d" % (M, K, N))


def test_workspace_errors():
    M, K, N = 4, 1024, 128
    d = wl.make_problem(M, K, N, seed=94)
    pw = pack_problem(d, N, K)
    A = to_dev(d["A"])
    B.w4a16_set_workspace(None)
    with pytest.raises(B.W4A16Error) as e:
        B.w4a16_gemm(A, pw, split_k=4, path=B.PATH_DECODE)
    assert e.value.code == -5
    small = torch.empty(B.WS_HEADER_BYTES + 1024, dtype=torch.uint8, device="cuda")
    B.w4a16_set_workspace(small[(-small.data_ptr()) % 256:][:B.WS_HEADER_BYTES + 256])
    with pytest.raises(B.W4A16Error) as e:
        B.w4a16_gemm(A, pw, split_k=4, path=B.PATH_DECODE)
    assert e.value.code == -5
    B.w4a16_set_workspace(None)
    # split_k = 1 needs none
    B.w4a16_gemm(A, pw, split_k=1, path=B.PATH_DECODE)
    torch.cuda.synchronize()


# Host result buffer: page-locked memory takes the kernel's stores directly (the device staging buffer is then
# left alone), ordinary pageable memory gets the result through the staging buffer and a copy.  Both on the
# warp-MMA kernel (M = 8) and the tcgen05 kernel (M = 40).
@pytest.mark.parametrize("pinned", [True, False])
@pytest.mark.parametrize("M", [8, 40])
def test_host_buffer_entry_point_matches_device_call(M, pinned):
    K, N = 1024, 256
    d = wl.make_problem(M, K, N, seed=95 + M)
    pw = pack_problem(d, N, K)
    ws = ensure_ws(M, N, K, 0)
    A_host = torch.from_numpy(d["A"].view(np.float16)).pin_memory()
    C_host = torch.zeros((M, N), dtype=torch.float16)
    if pinned:
        C_host = C_host.pin_memory()
    A_dev = torch.empty((M, K), dtype=torch.float16, device="cuda")
    C_dev = torch.zeros((M, N), dtype=torch.float16, device="cuda")
    for _ in range(2):
        B.w4a16_gemm_host(A_host, A_dev, pw, C_dev, C_host)
        torch.cuda.synchronize()
    C = B.w4a16_gemm(to_dev(d["A"]), pw)
    assert np.array_equal(C_host.numpy().view(np.uint16), c_bits(C))
    if not pinned:
        assert np.array_equal(c_bits(C_dev), c_bits(C))
    assert B.w4a16_device_status() == 0
    del ws


@pytest.mark.parametrize("M,split_k", [(1, 2), (5, 4), (8, 3), (16, 4), (12, 6)])
def test_cluster_exchange_and_workspace_exchange_give_the_same_bits(M, split_k):
    # Algorithm 1, Phase 3 in its two forms: w4a16_gemm on the warp-MMA path adds the slices of a tile
    # inside a thread-block cluster when each slice has a CTA of its own; w4a16_gemm_static_ws keeps
    # the workspace form (partial tiles, tickets, last arriver).  Both add in ascending K order, so
    # the outputs must agree bit for bit, and with the oracle within tolerance.
    K, N = 4096, 1024
    d = wl.make_problem(M, K, N, seed=600 + M)
    pw = pack_problem(d, N, K)
    A = to_dev(d["A"])
    ws = ensure_ws(M, N, K, split_k)
    got = B.w4a16_gemm(A, pw, split_k=split_k, path=B.PATH_DECODE)
    other = B.w4a16_gemm_static_ws(A, pw, split_k=split_k)
    torch.cuda.synchronize()
    assert B.w4a16_device_status() == 0
    assert np.array_equal(c_bits(got), c_bits(other))
    ref = oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, 128)
    assert_close(c_f64(got), ref, "M%d split %d" % (M, split_k))
    del ws


# The warp-MMA kernel brings a stage's activation rows either as one bulk copy per row (one batch row, or
# K < 512) or as one tensor copy of 8 or 16 rows x 512 k (rows past M and k past K read as zero): both
# forms at every edge -- K below, at and above one box, K not a multiple of the box, M at the block edges.
@pytest.mark.parametrize("K", [128, 384, 512, 640, 1024])
@pytest.mark.parametrize("M", [2, 7, 8, 9, 15, 16])
def test_activation_row_paths(M, K):
    N = 192
    d = wl.make_problem(M, K, N, seed=31 * M + K)
    ref = oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, 128)
    for split_k in (0, 1):
        C = _run(d, M, N, K, split_k, B.PATH_DECODE)
        assert_close(c_f64(C), ref, "decode M%d K%d S%d" % (M, K, split_k))
