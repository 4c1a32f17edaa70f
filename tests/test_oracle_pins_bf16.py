"""Pins of the oracle's BF16 functions (Section 1 names BF16 beside FP16 as the format the weights
are dequantized to) against things that are not the oracle: hand-derived encodings, torch's
bfloat16 conversion and arithmetic, exact rational arithmetic, the int64 closed form.  No GPU."""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from paper_2601_16536_b200 import workloads as wl

HERE = os.path.dirname(os.path.abspath(__file__))


def _bf16_to_f64(bits):
    b = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << 16
    return b.view(np.float32).astype(np.float64)


def test_bf16_golden_encodings():
    n = 0
    for line in open(os.path.join(HERE, "golden", "bf16_encodings.txt")):
        line = line.split("#")[0].strip() if line.lstrip().startswith("#") else line.strip()
        if not line:
            continue
        expr, bits = line.split("0x")[0].strip(), int(line.split("0x")[1].split()[0], 16)
        assert oracle.f64_to_bf16_rn(eval(expr)) == bits, expr
        n += 1
    assert n >= 20


def test_bf16_all_patterns_roundtrip_and_match_torch():
    bits = np.arange(65536, dtype=np.uint16)
    t = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).to(torch.float32).numpy()
    for b in range(65536):
        v = oracle.bf16_to_f32(b)
        if np.isnan(t[b]):
            assert np.isnan(v)
            continue
        assert v == t[b], hex(b)
        assert oracle.f64_to_bf16_rn(float(v)) == b, hex(b)


def test_f64_to_bf16_matches_torch_on_random_float32_and_halfway_points():
    r = np.random.Generator(np.random.PCG64(3))
    x = np.concatenate([r.standard_normal(4000).astype(np.float32) * np.float32(10.0) ** r.integers(-30, 30, 4000),
                        r.uniform(0.002, 0.02, 2000).astype(np.float32)]).astype(np.float32)
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = np.array([oracle.f64_to_bf16_rn(float(v)) for v in x], dtype=np.uint16)
    assert np.array_equal(got, want)
    # every halfway point between neighbouring positive normal values of one binade, and a hair either side
    for b in range(0x3F80, 0x4000):
        lo, hi = _bf16_to_f64([b])[0], _bf16_to_f64([b + 1])[0]
        mid = (lo + hi) / 2
        even = b if b % 2 == 0 else b + 1
        assert oracle.f64_to_bf16_rn(mid) == even
        assert oracle.f64_to_bf16_rn(np.nextafter(mid, 0)) == b
        assert oracle.f64_to_bf16_rn(np.nextafter(mid, 4)) == b + 1


def test_dequant_bf16_all_q_z_pairs_against_torch_bfloat16_arithmetic():
    # K = 128 * (number of scales): one group per scale; columns enumerate z; the rows of a group cycle through q
    r = np.random.Generator(np.random.PCG64(4))
    s_bits = np.concatenate([r.integers(0x0001, 0x7F80, 200, dtype=np.uint64).astype(np.uint16),
                             np.array([0x0001, 0x007F, 0x0080, 0x3C24, 0x3CA4, 0x7F7F], dtype=np.uint16)])
    G, N = len(s_bits), 16
    K = 128 * G
    q = (np.arange(K)[:, None] % 16 + np.zeros((1, N), dtype=np.int64)).astype(np.uint32)
    Wq = np.zeros((K // 8, N), dtype=np.uint32)
    for i in range(8):
        Wq |= q[i::8] << np.uint32(4 * i)
    S = np.repeat(s_bits[:, None], N, axis=1)
    Z = np.repeat(np.arange(N, dtype=np.uint8)[None, :], G, axis=0)
    got = oracle.dequant(Wq, S, Z, K, N, 128, bf16=True)
    d = torch.from_numpy((q.astype(np.int64) - np.repeat(Z, 128, axis=0).astype(np.int64)).astype(np.float32)).to(torch.bfloat16)
    s = torch.from_numpy(np.repeat(S, 128, axis=0).view(np.int16)).view(torch.bfloat16)
    want = (d * s).view(torch.int16).numpy().view(np.uint16)      # one BF16 multiply: exact product, one rounding
    assert np.array_equal(got, want)


@pytest.mark.parametrize("group", [32, 128])
def test_gemm_bf16_brute_force(group):
    M, K, N = 2, 256, 3
    d = wl.make_problem(M, K, N, seed=41, group=group, bf16=True)
    got = oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, group, bf16=True)
    want = np.zeros((M, N))
    for n in range(N):
        col = []
        for k in range(K):
            q = (int(d["Wq"][k // 8, n]) >> (4 * (k % 8))) & 15
            dz = torch.tensor(float(q - int(d["Z"][k // group, n])), dtype=torch.bfloat16)
            s = torch.from_numpy(d["S"][k // group, n:n + 1].view(np.int16)).view(torch.bfloat16)[0]
            col.append(Fraction(float(dz * s)))
        for m in range(M):
            want[m, n] = float(sum(Fraction(float(_bf16_to_f64(d["A"][m, k:k + 1])[0])) * col[k] for k in range(K)))
    assert np.allclose(got, want, rtol=1e-13, atol=1e-15)


def test_gemm_bf16_equals_float64_matmul_of_the_dequantized_matrix_and_differs_from_fp16():
    M, K, N = 3, 384, 40
    d = wl.make_problem(M, K, N, seed=42, bf16=True)
    W = _bf16_to_f64(oracle.dequant(d["Wq"], d["S"], d["Z"], K, N, 128, bf16=True))
    got = oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, 128, bf16=True)
    assert np.allclose(got, _bf16_to_f64(d["A"]) @ W, rtol=1e-12, atol=1e-13)
    # the same bit patterns read as FP16 are different numbers: the flag really selects the format
    as_f16 = oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, 128)
    assert not np.allclose(got, as_f16)


def test_gemm_int_bf16_closed_form():
    M, K, N = 3, 512, 5
    d = wl.make_exact_problem(M, K, N, seed=43, bf16=True)
    q = oracle.unpack(d["Wq"], K, N).astype(np.int64)
    k = np.arange(K)
    w = (q - d["Z"][k // 128].astype(np.int64)) * np.ldexp(1.0, d["E"][k // 128].astype(np.int64))
    exact = d["A_int"].astype(np.float64) @ w          # small integers times powers of two: exact in float64
    want = torch.from_numpy(exact.astype(np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = oracle.gemm_int(d["A_int"], d["Wq"], d["E"], d["Z"], M, N, K, 128, bf16=True)
    assert np.array_equal(got, want)
    ref = oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, 128, bf16=True)
    assert np.array_equal(ref, exact)
