"""Pins of the oracle's quantizer (Eq. 1, x_q = round(x / s) + z) against what the formula and the
mathematics fix, none of them the oracle itself: recovery of an exactly representable grid, the
error bound |x - s (q - z)| <= s / 2 inside the clamp range, monotonicity, ties to even, the
symmetric case, degenerate groups.  No GPU."""
import numpy as np
import pytest

import oracle


def _f16(bits):
    return np.asarray(bits, dtype=np.uint16).view(np.float16).astype(np.float64)


def _bits(x):
    return np.ascontiguousarray(np.asarray(x, dtype=np.float16)).view(np.uint16)


@pytest.mark.parametrize("group", [32, 64, 128])
def test_an_exact_grid_is_recovered(group):
    # x = (q0 - z0) * 2^e with every level 0..15 present in every group: max - min = 15 * 2^e, so s = 2^e
    # exactly, z = z0, and the codes come back unchanged
    K, N = 256, 5
    r = np.random.Generator(np.random.PCG64(group))
    G = K // group
    q0 = np.stack([np.concatenate([r.permutation(np.arange(group) % 16) for _ in range(G)]) for _ in range(N)], axis=1)
    z0 = r.integers(0, 16, size=(G, N))
    e = r.integers(-9, -3, size=(G, N))
    k = np.arange(K)
    x = (q0 - z0[k // group]) * np.ldexp(1.0, e[k // group])
    Wq, S, Z = oracle.quantize(_bits(x), K, N, group)
    assert np.array_equal(_f16(S), np.ldexp(1.0, e))
    assert np.array_equal(Z, z0)
    assert np.array_equal(oracle.unpack(Wq, K, N), q0)
    # and dequantization (Eq. 2) returns the very same weights
    assert np.array_equal(_f16(oracle.dequant(Wq, S, Z, K, N, group)), x)


@pytest.mark.parametrize("symmetric", [False, True])
def test_round_trip_error_is_at_most_half_a_step_and_codes_are_monotone(symmetric):
    K, N, group = 512, 7, 128
    r = np.random.Generator(np.random.PCG64(11))
    x = _f16(_bits(r.standard_normal((K, N)) * 0.05))
    Wq, S, Z = oracle.quantize(_bits(x), K, N, group, symmetric=symmetric)
    q = oracle.unpack(Wq, K, N).astype(np.int64)
    assert q.min() >= 0 and q.max() <= 15
    k = np.arange(K)
    s, z = _f16(S)[k // group], Z[k // group].astype(np.int64)
    if symmetric:
        assert np.all(Z == 8)
    back = (q - z) * s
    # inside the clamp range the reconstruction is within half a step (a hair more for the FP32 division)
    inside = (q > 0) & (q < 15)
    assert np.all(np.abs(back - x)[inside] <= 0.5 * s[inside] * (1 + 1e-6))
    # the clamped ends may be off by more, but never by more than one and a half steps here (s is the
    # range / 15 rounded to FP16, z is rounded to an integer)
    assert np.all(np.abs(back - x) <= 1.5 * s)
    # within a group and column, larger weights never get smaller codes
    for g in range(K // group):
        for n in range(N):
            xs, qs = x[g * group:(g + 1) * group, n], q[g * group:(g + 1) * group, n]
            order = np.argsort(xs, kind="stable")
            assert np.all(np.diff(qs[order]) >= 0)


def test_ties_round_to_even_and_the_clamp_holds():
    # one group, s = 1 exactly (min = -5, max = 10): z = 5; x = 0.5, 1.5, 2.5, -0.5 -> round(x) = 0, 2, 2, -0
    K, N, group = 32, 1, 32
    x = np.zeros((K, N))
    x[:6, 0] = [-5.0, 10.0, 0.5, 1.5, 2.5, -0.5]
    Wq, S, Z = oracle.quantize(_bits(x), K, N, group)
    assert _f16(S)[0, 0] == 1.0 and Z[0, 0] == 5
    q = oracle.unpack(Wq, K, N)[:, 0]
    assert list(q[:6]) == [0, 15, 5, 7, 7, 5]
    assert np.all(q[6:] == 5)                       # x = 0 maps to the zero point


def test_symmetric_uses_the_largest_magnitude_over_seven():
    K, N, group = 32, 2, 32
    x = np.zeros((K, N))
    x[0, 0], x[1, 0], x[2, 0] = -3.5, 1.0, 3.4999         # amax 3.5 -> s = 0.5: codes -7, 2, 7 (+8)
    x[0, 1], x[1, 1] = 7.0, -7.0                          # s = 1
    Wq, S, Z = oracle.quantize(_bits(x), K, N, group, symmetric=True)
    assert list(_f16(S)[0]) == [0.5, 1.0] and np.all(Z == 8)
    q = oracle.unpack(Wq, K, N)
    assert list(q[:3, 0]) == [1, 10, 15] and list(q[:2, 1]) == [15, 1]


def test_a_constant_group_gets_scale_one_and_stays_in_range():
    K, N, group = 64, 3, 32
    x = np.zeros((K, N))
    x[:32, 1] = 3.0          # constant non-zero group: max - min = 0
    x[32:, 2] = -40.0        # constant, far below what four bits reach with s = 1
    Wq, S, Z = oracle.quantize(_bits(x), K, N, group)
    assert np.all(_f16(S) == 1.0)
    q = oracle.unpack(Wq, K, N)
    assert np.all(q <= 15)
    assert Z[0, 0] == 0 and np.all(q[:32, 0] == 0)
    assert Z[0, 1] == 0 and np.all(q[:32, 1] == 3)           # z = clamp(round(-3)) = 0, q = 3 + 0
    assert Z[1, 2] == 15 and np.all(q[32:, 2] == 0)          # z = clamp(40) = 15, q = clamp(-40 + 15) = 0


def test_bf16_scales_are_representable_in_bf16():
    K, N, group = 128, 4, 64
    r = np.random.Generator(np.random.PCG64(12))
    x32 = (r.standard_normal((K, N)) * 0.1).astype(np.float32)
    bits = ((x32.view(np.uint32).astype(np.uint64) + 0x7FFF + ((x32.view(np.uint32) >> 16) & 1)) >> 16).astype(np.uint16)
    Wq, S, Z = oracle.quantize(bits, K, N, group, bf16=True)
    x = (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    s = (S.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    rng = np.array([[x[g * group:(g + 1) * group, n].max() - x[g * group:(g + 1) * group, n].min() for n in range(N)]
                    for g in range(K // group)])
    assert np.all(np.abs(s - rng / 15) <= rng / 15 * 2.0 ** -8)     # (max - min) / 15 rounded to 8 significant bits
    assert oracle.unpack(Wq, K, N).max() <= 15
