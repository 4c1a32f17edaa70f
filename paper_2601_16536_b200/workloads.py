"""Seeded synthetic inputs shaped like LLM decode / prefill layers.

This module only draws random numbers and lists shapes.  It holds none of the
method's arithmetic (no unpacking, no dequantization, no products): the CUDA
path and the CPU oracle both consume the arrays it returns.

Raw (boundary) layout of one problem  C[M,N] = A[M,K] . Dequant(W)[K,N]:

  A   uint16 [M, K]        FP16 bit patterns, row-major
  Wq  uint32 [K/8, N]      eight unsigned 4-bit values per word along K
  S   uint16 [K/group, N]  FP16 bit patterns of the scales
  Z   uint8  [K/group, N]  zero points, 0..15, one per byte

Every nibble of a uniformly random 32-bit word is uniform over 0..15, so the
words are drawn directly.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, Iterator, List, Tuple

import numpy as np

GROUP = 128


# (N, K) of the layers the paper measures (Figure 2 a-f; its "K = 16348" is read as 16384)
PAPER_SHAPES = ((1536, 6144), (2048, 8192), (2048, 10240), (4096, 16384), (4608, 10240), (7168, 18432))


@dataclass(frozen=True)
class Case:
    config: int       # 1..5, the benchmark configuration the case belongs to; 6 = the paper's own shapes
    name: str
    M: int
    K: int
    N: int
    seed: int
    a_sigma: float = 1.0
    outliers: bool = False   # 1 % of K columns of A scaled x20 (outlier channels)


def _cases() -> List[Case]:
    out: List[Case] = [Case(1, "decode_4096x4096", 1, 4096, 4096, 0)]
    for i, M in enumerate((1, 2, 4, 8, 16)):
        out.append(Case(2, "down_proj_decode", M, 11008, 4096, 2000 + i))
    for i, M in enumerate((1, 4, 16, 32)):
        out.append(Case(3, "extreme_k_decode", M, 28672, 8192, 3000 + i, 0.5, True))
    layers = (("qkv", 4096, 12288), ("o_proj", 4096, 4096),
              ("gate_up", 4096, 22016), ("down", 11008, 4096))
    i = 0
    for lname, K, N in layers:
        for M in (1, 16, 64):
            out.append(Case(4, lname, M, K, N, 4000 + i))
            i += 1
    for i, M in enumerate((256, 1024, 4096)):
        out.append(Case(5, "prefill_8192", M, 8192, 8192, 5000 + i))
    # the paper's own shape set (Section 4.1, Figure 2: six (N, K) pairs, batch sizes up to 256)
    i = 0
    for N, K in PAPER_SHAPES:
        for M in (1, 8, 64, 256):
            out.append(Case(6, "paper_N%d_K%d" % (N, K), M, K, N, 6000 + i))
            i += 1
    return out


CASES: Tuple[Case, ...] = tuple(_cases())


def cases_of(config: int) -> List[Case]:
    return [c for c in CASES if c.config == config]


def _f16_bits(x: np.ndarray) -> np.ndarray:
    return np.ascontiguousarray(x.astype(np.float16)).view(np.uint16)


def _bf16_bits(x: np.ndarray) -> np.ndarray:
    """Storage format of the drawn numbers only: float32 -> the nearest BF16 pattern (ties to even)."""
    b = np.ascontiguousarray(x.astype(np.float32)).view(np.uint32).astype(np.uint64)
    return ((b + 0x7FFF + ((b >> 16) & 1)) >> 16).astype(np.uint16)


def _bits16(x: np.ndarray, bf16: bool) -> np.ndarray:
    return _bf16_bits(x) if bf16 else _f16_bits(x)


SYM_ZERO = 8    # the zero point every weight of a symmetric format has


def draw_weights(K: int, N: int, seed: int, group: int = GROUP, symmetric: bool = False,
                 bf16: bool = False) -> Dict[str, np.ndarray]:
    """Wq, S, Z in the raw layout: q uniform 0..15, s ~ U[0.002, 0.02], z uniform 0..15 (all 8 for a
    symmetric format: the array is what a checker needs, the symmetric GPU path takes no Z at all).
    ``bf16`` stores the scales as BF16 instead of FP16 patterns."""
    G = K // group
    rq = np.random.Generator(np.random.PCG64([seed, 1]))
    rs = np.random.Generator(np.random.PCG64([seed, 2]))
    rz = np.random.Generator(np.random.PCG64([seed, 3]))
    Wq = rq.integers(0, 2 ** 32, size=(K // 8, N), dtype=np.uint64).astype(np.uint32)
    S = _bits16(rs.uniform(0.002, 0.02, size=(G, N)).astype(np.float32), bf16)
    Z = rz.integers(0, 16, size=(G, N), dtype=np.uint8)
    if symmetric:
        Z = np.full((G, N), SYM_ZERO, dtype=np.uint8)
    return {"Wq": Wq, "S": S, "Z": Z}


def draw_activations(M: int, K: int, seed: int, sigma: float = 1.0,
                     outliers: bool = False, bf16: bool = False) -> np.ndarray:
    """A ~ N(0, sigma); with ``outliers`` round(0.01 K) seeded columns are scaled x20."""
    ra = np.random.Generator(np.random.PCG64([seed, 0]))
    A = ra.standard_normal(size=(M, K), dtype=np.float32) * np.float32(sigma)
    if outliers:
        ro = np.random.Generator(np.random.PCG64([seed, 4]))
        cols = ro.permutation(K)[: int(round(0.01 * K))]
        A[:, cols] *= np.float32(20.0)
    return _bits16(A, bf16)


def make_case(case: Case, group: int = GROUP) -> Dict[str, np.ndarray]:
    d = draw_weights(case.K, case.N, case.seed, group)
    d["A"] = draw_activations(case.M, case.K, case.seed, case.a_sigma, case.outliers)
    return d


def make_problem(M: int, K: int, N: int, seed: int, group: int = GROUP,
                 sigma: float = 1.0, outliers: bool = False, symmetric: bool = False,
                 bf16: bool = False) -> Dict[str, np.ndarray]:
    d = draw_weights(K, N, seed, group, symmetric, bf16)
    d["A"] = draw_activations(M, K, seed, sigma, outliers, bf16)
    return d


def make_exact_problem(M: int, K: int, N: int, seed: int, group: int = GROUP,
                       e_lo: int = -8, e_hi: int = -4, symmetric: bool = False,
                       bf16: bool = False) -> Dict[str, np.ndarray]:
    """Inputs for which every product and partial sum is exactly representable:
    A in {-1, 0, 1}, scales 2**E with integer E in [e_lo, e_hi].
    Returns the raw arrays plus ``A_int`` (int8) and ``E`` (int8)."""
    G = K // group
    r = np.random.Generator(np.random.PCG64([seed, 7]))
    A_int = r.integers(-1, 2, size=(M, K), dtype=np.int8)
    E = r.integers(e_lo, e_hi + 1, size=(G, N), dtype=np.int8)
    Wq = r.integers(0, 2 ** 32, size=(K // 8, N), dtype=np.uint64).astype(np.uint32)
    Z = r.integers(0, 16, size=(G, N), dtype=np.uint8)
    if symmetric:
        Z = np.full((G, N), SYM_ZERO, dtype=np.uint8)
    S = _bits16(np.ldexp(np.float32(1.0), E.astype(np.int32)).astype(np.float32), bf16)
    A = _bits16(A_int.astype(np.float32), bf16)
    return {"A": A, "A_int": A_int, "Wq": Wq, "S": S, "Z": Z, "E": E}


def algorithmic_bytes(M: int, K: int, N: int, group: int = GROUP, symmetric: bool = False) -> int:
    """Bytes one call must move: packed weights + 16-bit scales + 4-bit zeros (none when symmetric) + A + C."""
    G = K // group
    return K * N // 2 + G * N * 2 + (0 if symmetric else G * N // 2) + 2 * M * K + 2 * M * N


def iter_cases(configs=(1, 2, 3, 4, 5)) -> Iterator[Case]:
    for c in CASES:
        if c.config in configs:
            yield c
