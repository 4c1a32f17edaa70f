"""GPU: stream ordering of the packed weights, and the bounded-wait status path.

The GEMM kernels may prefetch packed weights before the previous kernel of their stream has
finished (programmatic dependent launch), so the library has to order the first GEMM of a stream
after a w4a16_pack enqueued on that stream.  The status path (a bounded wait that runs out) is
exercised with the library's diagnostic kernel: nothing faults, the context stays usable.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2601_16536_b200 import binding as B
from paper_2601_16536_b200 import workloads as wl
from gpu_util import assert_close, c_bits, c_f64, ensure_ws, pack_problem, to_dev

pytestmark = pytest.mark.gpu


def test_pack_then_gemm_on_a_side_stream_with_another_stream_in_between():
    # pack on stream A, an unrelated GEMM on stream B, then the GEMM on stream A: the last one must
    # see the packed weights complete although a GEMM was launched elsewhere in between
    M, K, N = 4, 11008, 4096
    d = wl.make_problem(M, K, N, seed=3101)
    other = wl.make_problem(M, 1024, 256, seed=3102)
    ref = oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, 128)
    ws = ensure_ws(M, N, K, 0)
    pw_other = pack_problem(other, 256, 1024)
    A, A_other = to_dev(d["A"]), to_dev(other["A"])
    raw = [to_dev(d[k]) for k in ("Wq", "S", "Z")]
    torch.cuda.synchronize()
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    first = None
    for rep in range(4):
        with torch.cuda.stream(sa):
            # a long kernel in front so that the pack kernels are still pending when the GEMM is enqueued
            filler = torch.empty(64 << 20, dtype=torch.uint8, device="cuda")
            filler.fill_(rep)
            pw = B.w4a16_pack(raw[0], raw[1], raw[2], N, K)
        with torch.cuda.stream(sb):
            B.w4a16_gemm(A_other, pw_other, split_k=1)
        with torch.cuda.stream(sa):
            C = B.w4a16_gemm(A, pw)
            C2 = B.w4a16_gemm(A, pw)          # the second one may overlap its predecessor again
        torch.cuda.synchronize()
        assert B.w4a16_device_status() == 0
        assert_close(c_f64(C), ref, "first GEMM after pack, rep %d" % rep)
        assert np.array_equal(c_bits(C), c_bits(C2))
        if first is None:
            first = c_bits(C).copy()
        assert np.array_equal(c_bits(C), first)
        del pw, filler
    del ws


@pytest.mark.parametrize("path,M", [(B.PATH_DECODE, 8), (B.PATH_TILE, 32)])
def test_gemm_on_a_non_default_stream_matches_the_default_stream(path, M):
    K, N = 2304, 512
    d = wl.make_problem(M, K, N, seed=3200 + M)
    pw = pack_problem(d, N, K)
    A = to_dev(d["A"])
    ws = ensure_ws(M, N, K, (0, 3))
    want = B.w4a16_gemm(A, pw, split_k=3, path=path)
    torch.cuda.synchronize()
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        got = [B.w4a16_gemm(A, pw, split_k=3, path=path) for _ in range(3)]
    torch.cuda.synchronize()
    assert B.w4a16_device_status() == 0
    for g in got:
        assert np.array_equal(c_bits(g), c_bits(want))
    assert_close(c_f64(want), oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, 128), "stream")
    del ws


def test_a_wait_that_runs_out_is_reported_and_the_library_keeps_working():
    M, K, N = 8, 1152, 256
    d = wl.make_problem(M, K, N, seed=3300)
    pw = pack_problem(d, N, K)
    A = to_dev(d["A"])
    ws = ensure_ws(M, N, K, 3)
    before = c_bits(B.w4a16_gemm(A, pw, split_k=3, path=B.PATH_DECODE)).copy()
    torch.cuda.synchronize()
    assert B.w4a16_device_status() == 0
    B.w4a16_selftest_wait_timeout(1000)          # a barrier nobody arrives on, 1 ms limit
    torch.cuda.synchronize()                     # the kernel returned by itself
    assert B.w4a16_device_status() == 1          # bit 0: a barrier wait ran out ...
    assert B.w4a16_device_status() == 0          # ... and reading the word cleared it
    # the workspace (whose ticket counters the status call re-zeroed) and both kernels still work
    after = c_bits(B.w4a16_gemm(A, pw, split_k=3, path=B.PATH_DECODE))
    assert np.array_equal(before, after)
    tile = B.w4a16_gemm(A, pw, split_k=3, path=B.PATH_TILE)
    torch.cuda.synchronize()
    assert B.w4a16_device_status() == 0
    assert_close(c_f64(tile), oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, 128), "after timeout")
    with pytest.raises(B.W4A16Error):
        B.w4a16_selftest_wait_timeout(0)
    del ws
