"""ctypes front end of the CPU oracle (``w4a16_oracle.c``).

TEST INFRASTRUCTURE ONLY: the tests, ``__graft_entry__.smoke()`` and the
benchmark's CPU-baseline leg load this; the product package never does.  It
shares no code with the CUDA path.

Each function is the plain definition of paper Eq. 2,
``C = A . Dequant(W)``, ``Dequant(W) = s (W - z)``; see the C file's header for
the readings taken where the paper is silent.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "w4a16_oracle.c")
_LIB = os.path.join(_HERE, "libw4a16_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (``-O2 -fopenmp``); returns the library path."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + ".tmp.%d" % os.getpid()
    subprocess.check_call(
        ["gcc", "-O2", "-fopenmp", "-fno-fast-math", "-ffp-contract=off", "-std=c11",
         "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
    os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        vp, i = ctypes.c_void_p, ctypes.c_int
        L.orc_f16_to_f32.restype = ctypes.c_float
        L.orc_f16_to_f32.argtypes = [ctypes.c_uint16]
        L.orc_f64_to_f16_rn.restype = ctypes.c_uint16
        L.orc_f64_to_f16_rn.argtypes = [ctypes.c_double]
        L.orc_f32_to_f16_rn.restype = ctypes.c_uint16
        L.orc_f32_to_f16_rn.argtypes = [ctypes.c_float]
        L.orc_unpack.restype = None
        L.orc_unpack.argtypes = [vp, i, i, vp]
        L.orc_dequant.restype = None
        L.orc_dequant.argtypes = [vp, vp, vp, i, i, i, vp]
        L.orc_gemm.restype = None
        L.orc_gemm.argtypes = [vp, vp, vp, vp, i, i, i, i, vp]
        L.orc_gemm_cols.restype = None
        L.orc_gemm_cols.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, vp]
        L.orc_gemm_kslice.restype = None
        L.orc_gemm_kslice.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, vp]
        L.orc_gemm_int.restype = i
        L.orc_gemm_int.argtypes = [vp, vp, vp, vp, i, i, i, i, vp]
        L.orc_bf16_to_f32.restype = ctypes.c_float
        L.orc_bf16_to_f32.argtypes = [ctypes.c_uint16]
        L.orc_f64_to_bf16_rn.restype = ctypes.c_uint16
        L.orc_f64_to_bf16_rn.argtypes = [ctypes.c_double]
        L.orc_dequant_fmt.restype = None
        L.orc_dequant_fmt.argtypes = [vp, vp, vp, i, i, i, i, vp]
        L.orc_gemm_fmt.restype = None
        L.orc_gemm_fmt.argtypes = [vp, vp, vp, vp, i, i, i, i, i, vp]
        L.orc_gemm_int_fmt.restype = i
        L.orc_gemm_int_fmt.argtypes = [vp, vp, vp, vp, i, i, i, i, i, vp]
        L.orc_quantize.restype = None
        L.orc_quantize.argtypes = [vp, i, i, i, i, i, vp, vp, vp]
        L.orc_num_threads.restype = i
        L.orc_num_threads.argtypes = []
        _lib = L
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _chk(a, dtype, shape=None):
    a = np.ascontiguousarray(a)
    if a.dtype != np.dtype(dtype):
        raise TypeError("expected %s, got %s" % (np.dtype(dtype), a.dtype))
    if shape is not None and tuple(a.shape) != tuple(shape):
        raise ValueError("expected shape %s, got %s" % (shape, a.shape))
    return a


def f16_to_f32(bits: int) -> float:
    return float(lib().orc_f16_to_f32(int(bits) & 0xFFFF))


def f64_to_f16_rn(x: float) -> int:
    return int(lib().orc_f64_to_f16_rn(float(x)))


def bf16_to_f32(bits: int) -> float:
    return float(lib().orc_bf16_to_f32(int(bits) & 0xFFFF))


def f64_to_bf16_rn(x: float) -> int:
    return int(lib().orc_f64_to_bf16_rn(float(x)))


def unpack(Wq: np.ndarray, K: int, N: int) -> np.ndarray:
    """q[k, n] (uint8, [K, N]) from the raw words Wq uint32 [K/8, N]."""
    Wq = _chk(Wq, np.uint32, (K // 8, N))
    q = np.empty((K, N), dtype=np.uint8)
    lib().orc_unpack(_p(Wq), K, N, _p(q))
    return q


def dequant(Wq, S, Z, K: int, N: int, group: int = 128, bf16: bool = False) -> np.ndarray:
    """16-bit patterns (uint16, [K, N]) of rn16((q - z) * s); FP16, or BF16 with ``bf16``."""
    Wq = _chk(Wq, np.uint32, (K // 8, N))
    S = _chk(S, np.uint16, (K // group, N))
    Z = _chk(Z, np.uint8, (K // group, N))
    W16 = np.empty((K, N), dtype=np.uint16)
    if bf16:
        lib().orc_dequant_fmt(_p(Wq), _p(S), _p(Z), K, N, group, 1, _p(W16))
    else:
        lib().orc_dequant(_p(Wq), _p(S), _p(Z), K, N, group, _p(W16))
    return W16


def gemm(A, Wq, S, Z, M: int, N: int, K: int, group: int = 128, cols=None, bf16: bool = False) -> np.ndarray:
    """C_ref (float64, [M, N]) = sum_k A[m,k] * w16[k,n] in FP64.

    ``cols=(n0, n1)`` computes only those columns (the rest are NaN); ``bf16``: A, S and the
    dequantized weights are BF16 instead of FP16."""
    A = _chk(A, np.uint16, (M, K))
    Wq = _chk(Wq, np.uint32, (K // 8, N))
    S = _chk(S, np.uint16, (K // group, N))
    Z = _chk(Z, np.uint8, (K // group, N))
    if bf16:
        if cols is not None:
            raise ValueError("cols is not available for the BF16 format")
        C = np.empty((M, N), dtype=np.float64)
        lib().orc_gemm_fmt(_p(A), _p(Wq), _p(S), _p(Z), M, N, K, group, 1, _p(C))
        return C
    if cols is None:
        C = np.empty((M, N), dtype=np.float64)
        lib().orc_gemm(_p(A), _p(Wq), _p(S), _p(Z), M, N, K, group, _p(C))
    else:
        C = np.full((M, N), np.nan, dtype=np.float64)
        lib().orc_gemm_cols(_p(A), _p(Wq), _p(S), _p(Z), M, N, K, group,
                            int(cols[0]), int(cols[1]), _p(C))
    return C


def gemm_kslice(A, Wq, S, Z, M, N, K, group, k0, k1) -> np.ndarray:
    """Partial result C_i of one K-slice [k0, k1) (Algorithm 1, Phase 2), FP64."""
    A = _chk(A, np.uint16, (M, K))
    Wq = _chk(Wq, np.uint32, (K // 8, N))
    S = _chk(S, np.uint16, (K // group, N))
    Z = _chk(Z, np.uint8, (K // group, N))
    C = np.empty((M, N), dtype=np.float64)
    lib().orc_gemm_kslice(_p(A), _p(Wq), _p(S), _p(Z), M, N, K, group, k0, k1, _p(C))
    return C


def gemm_int(A_int, Wq, E, Z, M, N, K, group=128, bf16: bool = False) -> np.ndarray:
    """Exact case: integer A (int8), scales 2**E (int8 exponents); FP16 (or BF16) bits [M, N]."""
    A_int = _chk(A_int, np.int8, (M, K))
    Wq = _chk(Wq, np.uint32, (K // 8, N))
    E = _chk(E, np.int8, (K // group, N))
    Z = _chk(Z, np.uint8, (K // group, N))
    C = np.empty((M, N), dtype=np.uint16)
    rc = lib().orc_gemm_int_fmt(_p(A_int), _p(Wq), _p(E), _p(Z), M, N, K, group, 1 if bf16 else 0, _p(C))
    if rc != 0:
        raise ValueError("exponent range too wide for the exact oracle")
    return C


def quantize(W16, K: int, N: int, group: int = 128, symmetric: bool = False, bf16: bool = False):
    """Eq. 1 per (group, column): 16-bit weights [K, N] -> (Wq uint32 [K/8, N], S uint16 [K/group, N],
    Z uint8 [K/group, N]) in the raw layout."""
    W16 = _chk(W16, np.uint16, (K, N))
    Wq = np.empty((K // 8, N), dtype=np.uint32)
    S = np.empty((K // group, N), dtype=np.uint16)
    Z = np.empty((K // group, N), dtype=np.uint8)
    lib().orc_quantize(_p(W16), K, N, group, 1 if symmetric else 0, 1 if bf16 else 0, _p(Wq), _p(S), _p(Z))
    return Wq, S, Z


def epilogue(C_ref: np.ndarray, bias=None, act: str = "none") -> np.ndarray:
    """The optional step after the product (outside the paper's Algorithm 1), in FP64:
    y = act(C_ref + bias[n]) with act in {"none", "relu": max(x, 0), "silu": x / (1 + exp(-x))}."""
    y = np.array(C_ref, dtype=np.float64, copy=True)
    if bias is not None:
        y = y + np.asarray(bias, dtype=np.float64)[None, :]
    if act == "relu":
        y = np.maximum(y, 0.0)
    elif act == "silu":
        y = y / (1.0 + np.exp(-y))
    elif act != "none":
        raise ValueError(act)
    return y


def num_threads() -> int:
    return int(lib().orc_num_threads())
