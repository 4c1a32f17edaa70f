"""Pins for the CPU oracle: each check compares it with something that is not the oracle
(IEEE-754 encodings, numpy's float16, exact rational arithmetic, closed forms, invariants).

The operation is paper Eq. 2, C = A . Dequant(W), Dequant(W) = s (W - z); Algorithm 1 adds
"Dequantize to FP16" (Phase 1), Split-K partial sums (Phase 2) and sum + FP32->FP16 (Phase 3).
"""
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2601_16536_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _bits_to_f64(bits):
    return np.asarray(bits, dtype=np.uint16).view(np.float16).astype(np.float64)


# ---------------------------------------------------------------- FP16 conversions

def test_f16_golden_encodings():
    n = 0
    for line in open(os.path.join(GOLDEN, "fp16_encodings.txt")):
        line = line.split("#")[0].strip()
        if not line:
            continue
        v, b = line.split()
        assert oracle.f64_to_f16_rn(float.fromhex(v)) == int(b, 16), line
        n += 1
    assert n >= 20


def test_f16_all_patterns_roundtrip_and_match_numpy():
    L = oracle.lib()
    all_bits = np.arange(65536, dtype=np.uint16)
    ref = all_bits.view(np.float16).astype(np.float32)
    for b in range(65536):
        f = L.orc_f16_to_f32(b)
        r = float(ref[b])
        if np.isnan(r):
            assert np.isnan(f)
            continue
        assert f == r and np.signbit(f) == np.signbit(r), hex(b)
        assert L.orc_f64_to_f16_rn(f) == b, hex(b)


def test_f64_to_f16_matches_numpy_on_random_and_halfway_values():
    rng = np.random.default_rng(11)
    xs = [rng.standard_normal(20000) * s for s in (1e-7, 1e-5, 1e-3, 1.0, 100.0, 3e4, 7e4)]
    # exact halfway points between neighbouring finite binary16 values, and their neighbours
    pos = np.arange(0, 0x7C00, dtype=np.uint16).view(np.float16).astype(np.float64)
    mid = (pos[:-1] + pos[1:]) / 2
    xs += [mid, -mid, np.nextafter(mid, np.inf), np.nextafter(mid, -np.inf)]
    x = np.concatenate(xs)
    with np.errstate(over="ignore"):
        want = x.astype(np.float16).view(np.uint16)
    L = oracle.lib()
    got = np.array([L.orc_f64_to_f16_rn(float(v)) for v in x], dtype=np.uint16)
    assert np.array_equal(got, want)


# ---------------------------------------------------------------- unpack

def test_unpack_nibble_order_brute_force():
    # word 0x76543210: nibble i holds the value i, so q[8*kk + i, n] = i
    K, N = 16, 3
    Wq = np.empty((2, N), dtype=np.uint32)
    Wq[0, :] = 0x76543210
    Wq[1, :] = 0xFEDCBA98
    q = oracle.unpack(Wq, K, N)
    for n in range(N):
        assert list(q[:, n]) == list(range(16))


def test_unpack_matches_python_bit_arithmetic_on_random_words():
    rng = np.random.default_rng(5)
    K, N = 64, 7
    Wq = rng.integers(0, 2 ** 32, size=(K // 8, N), dtype=np.uint64).astype(np.uint32)
    q = oracle.unpack(Wq, K, N)
    for k in range(K):
        for n in range(N):
            assert q[k, n] == (int(Wq[k // 8, n]) >> (4 * (k % 8))) % 16
    # re-packing the unpacked nibbles gives the words back (bijection)
    re = np.zeros_like(Wq, dtype=np.uint64)
    for k in range(K):
        re[k // 8] |= q[k].astype(np.uint64) << np.uint64(4 * (k % 8))
    assert np.array_equal(re.astype(np.uint32), Wq)


# ---------------------------------------------------------------- dequant

def _all_qz_problem(s_bits):
    """K=128*len(s) rows... one group per scale; columns enumerate z; rows enumerate q."""
    G = len(s_bits)
    K, N = 128 * G, 16
    q = (np.arange(K)[:, None] % 16).astype(np.uint64) * np.ones((1, N), dtype=np.uint64)
    Wq = np.zeros((K // 8, N), dtype=np.uint64)
    for k in range(K):
        Wq[k // 8] |= q[k] << np.uint64(4 * (k % 8))
    Z = np.tile(np.arange(16, dtype=np.uint8), (G, 1))
    S = np.repeat(np.asarray(s_bits, dtype=np.uint16)[:, None], N, axis=1)
    return Wq.astype(np.uint32), S, Z, K, N, q.astype(np.int32)


def test_dequant_all_q_z_pairs_against_numpy_float16():
    rng = np.random.default_rng(3)
    # sampled FP16 scales: subnormal, tiny, the benchmark range, large, negative
    s_bits = np.concatenate([
        np.array([0x0001, 0x0003, 0x03FF, 0x0400, 0x3C00, 0x7BFF, 0x77FF, 0x211F, 0x9C00], np.uint16),
        rng.integers(0, 0x7C00, size=200).astype(np.uint16),
        rng.uniform(0.002, 0.02, size=300).astype(np.float16).view(np.uint16),
    ])
    Wq, S, Z, K, N, q = _all_qz_problem(s_bits)
    got = oracle.dequant(Wq, S, Z, K, N, 128)
    s32 = np.repeat(S.view(np.float16).astype(np.float32), 128, axis=0)
    z32 = np.repeat(Z.astype(np.int32), 128, axis=0)
    with np.errstate(over="ignore"):
        # (q - z) has <= 4 significant bits and s 11, so the float32 product is exact;
        # numpy's float32 -> float16 cast is round-to-nearest-even
        want = ((q - z32).astype(np.float32) * s32).astype(np.float16).view(np.uint16)
    # +0 vs -0: (q - z) = 0 times a negative s is -0 in IEEE; compare values and bits elsewhere
    assert np.array_equal(got, want)


def test_dequant_q_equals_z_gives_zero():
    d = wl.draw_weights(256, 64, seed=9)
    K, N = 256, 64
    Z = np.repeat(np.arange(2, dtype=np.uint8)[:, None] * 7 + 3, N, axis=1)  # z = 3, 10
    # build words whose every nibble equals z of its group
    Wq = np.empty((K // 8, N), dtype=np.uint32)
    Wq[:16] = 0x33333333
    Wq[16:] = 0xAAAAAAAA
    got = oracle.dequant(Wq, d["S"], Z, K, N, 128)
    assert np.all(got == 0)


def test_dequant_subtracts_before_multiplying():
    # s*(q - z) and s*q - s*z differ after FP16 rounding for some inputs; the oracle must be
    # the former (Eq. 2 writes s(W - z)).  Find such an input and check which one it matches.
    s = np.float16(0.01153)
    found = False
    for q in range(16):
        for z in range(16):
            a = np.float16(np.float32(q - z) * np.float32(s))
            b = np.float16(np.float16(np.float32(q) * np.float32(s)) - np.float16(np.float32(z) * np.float32(s)))
            if a != b:
                found = True
                Wq = np.full((16, 1), q * 0x11111111, dtype=np.uint32)
                S = np.full((1, 1), s.view(np.uint16), dtype=np.uint16)
                Z = np.full((1, 1), z, dtype=np.uint8)
                got = oracle.dequant(Wq, S, Z, 128, 1, 128)
                assert np.all(got == a.view(np.uint16))
    assert found


# ---------------------------------------------------------------- gemm

def _exact_rational_gemm(A, Wq, S, Z, M, N, K, group):
    """Second, independent implementation in the test: exact Fractions, w16 via numpy float16."""
    out = [[Fraction(0)] * N for _ in range(M)]
    for n in range(N):
        col = []
        for k in range(K):
            q = (int(Wq[k // 8, n]) >> (4 * (k % 8))) & 15
            z = int(Z[k // group, n])
            s = np.uint16(S[k // group, n]).view(np.float16)
            w16 = np.float16(np.float32(q - z) * np.float32(s))
            col.append(Fraction(float(w16)))
        for m in range(M):
            acc = Fraction(0)
            for k in range(K):
                acc += Fraction(float(np.uint16(A[m, k]).view(np.float16))) * col[k]
            out[m][n] = acc
    return np.array([[float(v) for v in row] for row in out], dtype=np.float64)


@pytest.mark.parametrize("M,K,N", [(1, 128, 8), (3, 256, 5), (2, 384, 3)])
def test_gemm_brute_force_tiny_shapes(M, K, N):
    d = wl.make_problem(M, K, N, seed=100 + M)
    got = oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, 128)
    want = _exact_rational_gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, 128)
    assert np.allclose(got, want, rtol=1e-13, atol=1e-15)


def test_gemm_matches_numpy_float64_matmul_of_dequantized_weights():
    M, K, N = 5, 512, 192
    d = wl.make_problem(M, K, N, seed=21)
    W16 = oracle.dequant(d["Wq"], d["S"], d["Z"], K, N, 128)
    want = _bits_to_f64(d["A"]) @ _bits_to_f64(W16)
    got = oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, 128)
    assert np.allclose(got, want, rtol=1e-12, atol=1e-13)


def test_gemm_operand_orientation_is_not_transposed():
    # A = e_m e_k^T picks out exactly w16[k, n]: catches swapped / transposed indices.
    M, K, N = 2, 256, 64
    d = wl.make_problem(M, K, N, seed=22)
    A = np.zeros((M, K), dtype=np.uint16)
    A[0, 5] = 0x3C00      # 1.0
    A[1, 200] = 0x4000    # 2.0
    W16 = _bits_to_f64(oracle.dequant(d["Wq"], d["S"], d["Z"], K, N, 128))
    got = oracle.gemm(A, d["Wq"], d["S"], d["Z"], M, N, K, 128)
    assert np.array_equal(got[0], W16[5])
    assert np.array_equal(got[1], 2.0 * W16[200])


def test_gemm_exact_closed_form_s1_z8():
    # s = 1, z = 8, A in {-1,0,1}: C = sum_k a (q - 8) is an integer; FP64 must hold it exactly,
    # and it must equal an int64 numpy computation.
    M, K, N = 4, 1024, 96
    d = wl.make_exact_problem(M, K, N, seed=31, e_lo=0, e_hi=0)
    d["Z"][:] = 8
    q = oracle.unpack(d["Wq"], K, N).astype(np.int64)
    want = d["A_int"].astype(np.int64) @ (q - 8)
    got = oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, 128)
    assert np.array_equal(got, want.astype(np.float64))
    c16 = oracle.gemm_int(d["A_int"], d["Wq"], d["E"], d["Z"], M, N, K, 128)
    with np.errstate(over="ignore"):
        assert np.array_equal(c16, want.astype(np.float64).astype(np.float16).view(np.uint16))


def test_gemm_int_equals_fp64_oracle_rounded_with_power_of_two_scales():
    M, K, N = 3, 2048, 128
    d = wl.make_exact_problem(M, K, N, seed=32)
    c64 = oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, 128)
    c16 = oracle.gemm_int(d["A_int"], d["Wq"], d["E"], d["Z"], M, N, K, 128)
    # FP64 is exact here (all terms multiples of 2^-8, |sum| << 2^44), so one rounding each
    assert np.array_equal(c16, c64.astype(np.float16).view(np.uint16))
    # and against an independent int64 numpy evaluation
    q = oracle.unpack(d["Wq"], K, N).astype(np.int64)
    z = np.repeat(d["Z"].astype(np.int64), 128, axis=0)
    sc = np.repeat(np.int64(1) << (d["E"].astype(np.int64) + 8), 128, axis=0)   # units of 2^-8
    want = (d["A_int"].astype(np.int64) @ ((q - z) * sc)).astype(np.float64) / 256.0
    assert np.array_equal(c64, want)


def test_gemm_q_equals_z_gives_zero():
    M, K, N = 2, 256, 64
    d = wl.make_problem(M, K, N, seed=41)
    Z = np.empty((2, N), dtype=np.uint8)
    Z[0], Z[1] = 5, 12
    Wq = np.empty((K // 8, N), dtype=np.uint32)
    Wq[:16], Wq[16:] = 0x55555555, 0xCCCCCCCC
    got = oracle.gemm(d["A"], Wq, d["S"], Z, M, N, K, 128)
    assert np.all(got == 0.0)


def test_gemm_doubling_scales_doubles_result_exactly():
    M, K, N = 2, 512, 64
    d = wl.make_problem(M, K, N, seed=42)
    S2 = (d["S"].view(np.float16) * np.float16(2)).view(np.uint16)
    c1 = oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, 128)
    c2 = oracle.gemm(d["A"], d["Wq"], S2, d["Z"], M, N, K, 128)
    assert np.array_equal(c2, 2.0 * c1)


def test_gemm_per_group_linearity():
    # C = sum_g C_g where C_g keeps group g and sets q == z in all others.
    M, K, N = 2, 512, 64
    G = K // 128
    d = wl.make_problem(M, K, N, seed=43)
    full = oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, 128)
    total = np.zeros_like(full)
    for g in range(G):
        Wq = (d["Z"].astype(np.uint32) * np.uint32(0x11111111))          # every nibble = z
        Wq = np.repeat(Wq, 16, axis=0)
        Wq[g * 16:(g + 1) * 16] = d["Wq"][g * 16:(g + 1) * 16]
        total += oracle.gemm(d["A"], Wq, d["S"], d["Z"], M, N, K, 128)
    assert np.allclose(total, full, rtol=1e-12, atol=1e-13)


def test_gemm_invariant_under_permuting_groups_of_k():
    M, K, N = 2, 512, 64
    d = wl.make_problem(M, K, N, seed=44)
    perm = np.array([2, 0, 3, 1])
    A = d["A"].reshape(M, 4, 128)[:, perm].reshape(M, K)
    Wq = d["Wq"].reshape(4, 16, N)[perm].reshape(K // 8, N)
    c1 = oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, 128)
    c2 = oracle.gemm(np.ascontiguousarray(A), np.ascontiguousarray(Wq),
                     np.ascontiguousarray(d["S"][perm]), np.ascontiguousarray(d["Z"][perm]),
                     M, N, K, 128)
    assert np.allclose(c1, c2, rtol=1e-12, atol=1e-13)


def test_split_k_partials_sum_to_the_whole():
    # Phase 3: C = sum_{i<S} C_i, with whole-group slices of unequal size (5 groups, S = 3)
    M, K, N = 3, 640, 64
    d = wl.make_problem(M, K, N, seed=45)
    full = oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, 128)
    bounds = [0, 256, 512, 640]
    parts = [oracle.gemm_kslice(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, 128, bounds[i], bounds[i + 1])
             for i in range(3)]
    assert np.allclose(sum(parts), full, rtol=1e-12, atol=1e-13)
    W16 = _bits_to_f64(oracle.dequant(d["Wq"], d["S"], d["Z"], K, N, 128))
    a = _bits_to_f64(d["A"])
    assert np.allclose(parts[1], a[:, 256:512] @ W16[256:512], rtol=1e-12, atol=1e-13)


def test_gemm_cols_subset_equals_full():
    M, K, N = 2, 256, 64
    d = wl.make_problem(M, K, N, seed=46)
    full = oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, 128)
    part = oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, 128, cols=(10, 20))
    assert np.array_equal(part[:, 10:20], full[:, 10:20])
    assert np.all(np.isnan(part[:, :10])) and np.all(np.isnan(part[:, 20:]))
