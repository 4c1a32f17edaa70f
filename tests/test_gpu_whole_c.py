"""GPU parity on the WHOLE output at the benchmark's full sizes (every row, every column, element by
element against the FP64 oracle of Eq. 2), in the launch configuration bench.py times (automatic
path, automatic split): one case per (K, N) of configs 1-4 at the largest M <= 16, the paper's own
shapes (Section 4.1) at M = 1, and for the prefill config seeded rows over all N -- the first and
last row of batch tiles among them -- so that a fault confined to one column tile, one CTA's chunk
or one Split-K slice cannot pass."""
import numpy as np
import pytest
import torch

import oracle
from paper_2601_16536_b200 import binding as B
from paper_2601_16536_b200 import workloads as wl
from gpu_util import assert_close, c_f64, ensure_ws, pack_problem, to_dev

pytestmark = pytest.mark.gpu


def _largest_small_m_per_layer():
    best = {}
    for c in wl.CASES:
        if c.config in (1, 2, 3, 4) and c.M <= 16:
            key = (c.config, c.K, c.N)
            if key not in best or c.M > best[key].M:
                best[key] = c
    return list(best.values()) + [c for c in wl.cases_of(6) if c.M == 1]


@pytest.mark.parametrize("case", _largest_small_m_per_layer(),
                         ids=lambda c: "cfg%d-%s-M%d" % (c.config, c.name, c.M))
def test_whole_output_matches_the_oracle(case):
    M, K, N = case.M, case.K, case.N
    d = wl.make_case(case)
    pw = pack_problem(d, N, K)
    ws = ensure_ws(M, N, K, 0)
    C = B.w4a16_gemm(to_dev(d["A"]), pw)
    torch.cuda.synchronize()
    assert B.w4a16_device_status() == 0
    ref = oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, 128)
    assert_close(c_f64(C), ref, "cfg%d %s M%d whole C" % (case.config, case.name, M))
    del ws


@pytest.mark.parametrize("M", [256, 1024, 4096])
def test_prefill_config_seeded_rows_over_all_columns(M):
    case = [c for c in wl.cases_of(5) if c.M == M][0]
    d = wl.make_case(case)
    K, N = case.K, case.N
    pw = pack_problem(d, N, K)
    ws = ensure_ws(M, N, K, 0)
    C = B.w4a16_gemm(to_dev(d["A"]), pw)
    torch.cuda.synchronize()
    assert B.w4a16_device_status() == 0
    rng = np.random.Generator(np.random.PCG64([case.seed, 99]))
    edges = [r for t in range(0, M, 256) for r in (t, t + 127, t + 128, t + 255)][:24]
    rows = sorted(set(edges) | set(int(r) for r in rng.choice(M, size=64 - len(set(edges)), replace=False)))
    A_rows = np.ascontiguousarray(d["A"][rows])
    ref = oracle.gemm(A_rows, d["Wq"], d["S"], d["Z"], len(rows), N, K, 128)     # these rows, every column
    got = c_f64(C)[rows]
    assert_close(got, ref, "prefill M%d, %d rows over all N" % (M, len(rows)))
    del ws
