"""GPU: w4a16_gemm_static_ws, the entry point for callers that cannot allocate device memory.

Such callers (a serving runtime that fixed its memory plan at start-up, a plug-in living in another
framework's pool, a latency-bound loop that must never enter the allocator) cannot give the library
a Split-K workspace.  The entry point therefore keeps its partial tiles and ticket counters in an
array compiled into the library.  Here it is called through the C ABI twice in a row -- the second
call finds the first call's leftovers in that array -- and each result is compared with what the
ordinary entry point returns for the same inputs with a caller-owned workspace.

This file sorts last on purpose: a run that stops at the first failure has then already run every
other test.  It builds its own inputs and registers its own workspace, so it also passes alone.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2601_16536_b200 import binding as B
from paper_2601_16536_b200 import workloads as wl
from gpu_util import assert_close, c_bits, c_f64, ensure_ws, pack_problem, to_dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("M,K,N,split_k", [(1, 4096, 1024, 0), (16, 2304, 512, 0), (5, 1152, 256, 3)])
def test_static_scratch_matches_the_workspace_entry_point_twice(M, K, N, split_k):
    d = wl.make_problem(M, K, N, seed=4242 + M)
    pw = pack_problem(d, N, K)
    A = to_dev(d["A"])
    ws = ensure_ws(M, N, K, split_k)
    want = B.w4a16_gemm(A, pw, split_k=split_k, path=B.PATH_DECODE)
    torch.cuda.synchronize()
    B.w4a16_set_workspace(None)        # from here on the library has no caller-owned scratch
    del ws
    ref = oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, 128)
    C = torch.empty((M, N), dtype=torch.float16, device="cuda")
    results = []
    for call in range(2):
        C.fill_(float("nan"))
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        B.w4a16_gemm_static_ws(A, pw, C, split_k=split_k)
        torch.cuda.synchronize()
        if call == 1:
            # the entry point's one promise: no device memory is taken.  (The first call of a process may
            # load the kernel's code; the second finds everything in place.)
            assert torch.cuda.mem_get_info()[0] == free_before
        assert B.w4a16_device_status() == 0
        # same tolerances as the other GEMM parity tests, against the existing entry point ...
        assert_close(c_f64(C), c_f64(want), "static scratch vs workspace, call %d" % call)
        # ... and against the oracle
        assert_close(c_f64(C), ref, "static scratch vs oracle, call %d" % call)
        results.append(c_bits(C).copy())
    assert np.array_equal(results[0], results[1])


def test_whole_tile_schedules_need_no_scratch_however_wide():
    # N = 128256 (2004 column tiles): the library deals whole tiles, which leave no partial tiles and draw no
    # tickets, so the shape runs although 2004 partial-tile slots would not fit the built-in array
    M, K, N = 1, 1024, 128256
    d = wl.make_problem(M, K, N, seed=11)
    pw = pack_problem(d, N, K)
    A = to_dev(d["A"])
    ref = oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, 128)
    for split_k in (0, 1):
        C = B.w4a16_gemm_static_ws(A, pw, split_k=split_k)
        torch.cuda.synchronize()
        assert B.w4a16_device_status() == 0
        assert_close(c_f64(C), ref, "wide N, split_k %d" % split_k)


def test_static_scratch_rejects_what_does_not_fit():
    # 64 column tiles x 86 splits of 16-row partial tiles need far more than the built-in array
    M, K, N = 16, 11008, 4096
    d = wl.make_problem(M, K, N, seed=7)
    pw = pack_problem(d, N, K)
    with pytest.raises(B.W4A16Error) as e:
        B.w4a16_gemm_static_ws(to_dev(d["A"]), pw, split_k=86)
    assert e.value.code == -5
