"""Pins of the CPU oracle for the quantization-format variants: groups of 32 and 64 along K and the
symmetric case of Eq. 1 (zero point fixed; 8 for the unsigned nibbles).  The oracle takes `group`
and Z as parameters; here those parameters are checked against things that are not the oracle:
exact rational arithmetic on tiny shapes, numpy float16, a float64 matmul and the int64 closed form.
No GPU."""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2601_16536_b200 import workloads as wl


def _f16(bits):
    return np.asarray(bits, dtype=np.uint16).view(np.float16).astype(np.float64)


def _rational_gemm(A, Wq, S, Z, M, N, K, group):
    out = np.zeros((M, N))
    for n in range(N):
        col = []
        for k in range(K):
            q = (int(Wq[k // 8, n]) >> (4 * (k % 8))) & 15
            w16 = np.float16(np.float32(q - int(Z[k // group, n])) * np.float32(np.uint16(S[k // group, n]).view(np.float16)))
            col.append(Fraction(float(w16)))
        for m in range(M):
            out[m, n] = float(sum(Fraction(float(np.uint16(A[m, k]).view(np.float16))) * col[k] for k in range(K)))
    return out


@pytest.mark.parametrize("group", [32, 64])
@pytest.mark.parametrize("symmetric", [False, True])
def test_gemm_brute_force_small_groups(group, symmetric):
    M, K, N = 2, 256, 4
    d = wl.make_problem(M, K, N, seed=500 + group, group=group, symmetric=symmetric)
    assert d["S"].shape == (K // group, N) and d["Z"].shape == (K // group, N)
    if symmetric:
        assert np.all(d["Z"] == 8)
    got = oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, group)
    want = _rational_gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, group)
    assert np.allclose(got, want, rtol=1e-13, atol=1e-15)


@pytest.mark.parametrize("group", [32, 64, 128])
def test_dequant_uses_the_scale_and_zero_of_the_right_group(group):
    # every group gets its own power-of-two scale and its own zero point: w = (q - z_g) * 2^e_g exactly,
    # so a group index off by one (or a group size of 128 used for all) changes the result
    K, N = 256, 3
    G = K // group
    r = np.random.Generator(np.random.PCG64(group))
    Wq = r.integers(0, 2 ** 32, size=(K // 8, N), dtype=np.uint64).astype(np.uint32)
    e = np.arange(G)[:, None] - 6 + np.zeros((1, N), dtype=np.int64)
    S = np.ldexp(np.float32(1), e.astype(np.int32)).astype(np.float16).view(np.uint16)
    Z = ((np.arange(G)[:, None] * 5 + np.arange(N)[None, :]) % 16).astype(np.uint8)
    got = _f16(oracle.dequant(Wq, S, Z, K, N, group))
    q = oracle.unpack(Wq, K, N).astype(np.int64)
    k = np.arange(K)
    want = (q - Z[k // group].astype(np.int64)) * np.ldexp(1.0, e[k // group])
    assert np.array_equal(got, want)


@pytest.mark.parametrize("group", [32, 64])
def test_gemm_equals_float64_matmul_of_the_dequantized_matrix(group):
    M, K, N = 4, 384, 70
    d = wl.make_problem(M, K, N, seed=77, group=group)
    W16 = _f16(oracle.dequant(d["Wq"], d["S"], d["Z"], K, N, group))
    got = oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, group)
    assert np.allclose(got, _f16(d["A"]) @ W16, rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("group", [32, 64, 128])
def test_symmetric_closed_form(group):
    # Eq. 1's symmetric case: z is the same for every weight.  With s = 1 and A = +-1/0 the product is the
    # integer sum_k a_k (q_k - 8); the int64 oracle and an independent numpy evaluation must agree.
    M, K, N = 3, 256, 6
    d = wl.make_exact_problem(M, K, N, seed=9, group=group, e_lo=0, e_hi=0, symmetric=True)
    q = oracle.unpack(d["Wq"], K, N).astype(np.int64)
    want = d["A_int"].astype(np.int64) @ (q - 8)
    got = oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, group)
    assert np.array_equal(got, want.astype(np.float64))
    bits = oracle.gemm_int(d["A_int"], d["Wq"], d["E"], d["Z"], M, N, K, group)
    assert np.array_equal(bits, want.astype(np.float16).view(np.uint16))


def test_a_group_of_32_is_not_a_group_of_128_with_repeated_scales_shifted():
    # the same scale/zero arrays read with the wrong group size give a different product
    M, K, N = 1, 256, 2
    d = wl.make_problem(M, K, N, seed=5, group=32)
    right = oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, 32)
    wrong = oracle.gemm(d["A"], d["Wq"], d["S"][:2], d["Z"][:2], M, N, K, 128)
    assert not np.allclose(right, wrong)


def test_epilogue_definitions():
    x = np.linspace(-6, 6, 25)[None, :]
    b = np.arange(25, dtype=np.float64) / 10
    assert np.array_equal(oracle.epilogue(x), x)
    assert np.array_equal(oracle.epilogue(x, b), x + b)
    relu = oracle.epilogue(x, None, "relu")
    assert np.all(relu >= 0) and np.array_equal(relu[x > 0], x[x > 0]) and np.all(relu[x <= 0] == 0)
    silu = oracle.epilogue(x, None, "silu")
    # silu(x) - silu(-x) = x,  silu(0) = 0,  silu(x) -> x for large x,  silu(1) = 1 / (1 + e^-1)
    assert np.allclose(silu - silu[:, ::-1], x, atol=1e-15)
    assert silu[0, 12] == 0.0 and abs(silu[0, -1] - 6.0) < 0.02
    assert abs(float(oracle.epilogue(np.array([[1.0]]), None, "silu")[0, 0]) - 0.7310585786300049) < 1e-15
    # bias is added before the activation
    assert np.array_equal(oracle.epilogue(np.array([[-1.0]]), [2.0], "relu"), [[1.0]])
