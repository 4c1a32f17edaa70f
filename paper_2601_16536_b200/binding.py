"""Thin ctypes binding over ``libw4a16.so`` (the C ABI of ``include/w4a16.h``).

Argument marshalling only: tensors are passed as raw device pointers, the stream as
the current ``torch.cuda`` stream's handle.  Every step of the computation runs in the
library's CUDA kernels.  There is no fallback: if the library is missing or a call
returns an error code, this raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libw4a16.so")

PATH_AUTO, PATH_SIMPLE, PATH_DECODE, PATH_TILE = 0, 1, 2, 3
FLAG_SYMMETRIC, FLAG_BF16 = 1, 2
ACT_NONE, ACT_RELU, ACT_SILU = 0, 1, 2
GROUP = 128
WS_HEADER_BYTES = 16384 + 131072   # W4A16_WORKSPACE_HEADER_BYTES

EXPORTS = (
    "w4a16_strerror", "w4a16_packed_wq_bytes", "w4a16_packed_s_bytes", "w4a16_packed_z_bytes",
    "w4a16_workspace_bytes", "w4a16_set_workspace", "w4a16_choose_split_k",
    "w4a16_choose_split_k_ex", "w4a16_choose_path", "w4a16_pack", "w4a16_dequant", "w4a16_gemm", "w4a16_gemm_ex",
    "w4a16_gemm_host", "w4a16_gemm_static_ws", "w4a16_device_status", "w4a16_selftest_wait_timeout",
    "w4a16_pack_fmt", "w4a16_dequant_fmt", "w4a16_gemm_fmt", "w4a16_quantize",
)

_lib = None


class W4A16Error(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__("%s failed: %d (%s)" % (what, code, strerror(code)))


def load():
    """Load the compiled library; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            "libw4a16.so is missing at %s: build it with `python -m paper_2601_16536_b200.build` "
            "(there is no CPU or PyTorch fallback)" % LIB_PATH)
    L = ctypes.CDLL(LIB_PATH)
    vp, i, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    L.w4a16_strerror.restype = ctypes.c_char_p
    L.w4a16_strerror.argtypes = [i]
    for name in ("w4a16_packed_wq_bytes", "w4a16_packed_s_bytes", "w4a16_packed_z_bytes"):
        getattr(L, name).restype = sz
        getattr(L, name).argtypes = [i, i, i]
    L.w4a16_workspace_bytes.restype = sz
    L.w4a16_workspace_bytes.argtypes = [i, i, i, i, i]
    L.w4a16_set_workspace.restype = i
    L.w4a16_set_workspace.argtypes = [vp, sz]
    L.w4a16_choose_split_k.restype = i
    L.w4a16_choose_split_k.argtypes = [i, i, i, i]
    L.w4a16_choose_path.restype = i
    L.w4a16_choose_path.argtypes = [i, i, i, i]
    L.w4a16_choose_split_k_ex.restype = i
    L.w4a16_choose_split_k_ex.argtypes = [i, i, i, i, i]
    L.w4a16_pack.restype = i
    L.w4a16_pack.argtypes = [vp, vp, vp, vp, vp, vp, i, i, i, vp]
    L.w4a16_dequant.restype = i
    L.w4a16_dequant.argtypes = [vp, vp, vp, vp, i, i, i, vp]
    L.w4a16_gemm.restype = i
    L.w4a16_gemm.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, i, vp]
    L.w4a16_gemm_ex.restype = i
    L.w4a16_gemm_ex.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, i, i, vp]
    L.w4a16_gemm_host.restype = i
    L.w4a16_gemm_host.argtypes = [vp, vp, vp, vp, vp, vp, vp, i, i, i, i, i, vp]
    L.w4a16_gemm_static_ws.restype = i
    L.w4a16_gemm_static_ws.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, i, vp]
    L.w4a16_pack_fmt.restype = i
    L.w4a16_pack_fmt.argtypes = [vp, vp, vp, vp, vp, vp, i, i, i, i, vp]
    L.w4a16_dequant_fmt.restype = i
    L.w4a16_dequant_fmt.argtypes = [vp, vp, vp, vp, i, i, i, i, vp]
    L.w4a16_gemm_fmt.restype = i
    L.w4a16_gemm_fmt.argtypes = [vp, vp, vp, vp, vp, vp, i, i, i, i, i, i, i, i, vp]
    L.w4a16_quantize.restype = i
    L.w4a16_quantize.argtypes = [vp, vp, vp, vp, i, i, i, i, vp]
    L.w4a16_selftest_wait_timeout.restype = i
    L.w4a16_selftest_wait_timeout.argtypes = [ctypes.c_uint, vp]
    L.w4a16_device_status.restype = i
    L.w4a16_device_status.argtypes = [ctypes.POINTER(ctypes.c_int)]
    _lib = L
    return L


def strerror(code: int) -> str:
    return load().w4a16_strerror(int(code)).decode()


def _check(rc: int, what: str):
    if rc != 0:
        raise W4A16Error(rc, what)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t: Optional[torch.Tensor]) -> int:
    return 0 if t is None else t.data_ptr()


# ------------------------------------------------------------------ sizes / heuristics
def w4a16_packed_wq_bytes(N: int, K: int, group: int = GROUP) -> int:
    return load().w4a16_packed_wq_bytes(N, K, group)


def w4a16_packed_s_bytes(N: int, K: int, group: int = GROUP) -> int:
    return load().w4a16_packed_s_bytes(N, K, group)


def w4a16_packed_z_bytes(N: int, K: int, group: int = GROUP) -> int:
    return load().w4a16_packed_z_bytes(N, K, group)


def w4a16_workspace_bytes(M: int, N: int, K: int, group: int = GROUP, split_k: int = 0) -> int:
    return load().w4a16_workspace_bytes(M, N, K, group, split_k)


def w4a16_choose_split_k(M: int, N: int, K: int, group: int = GROUP, path: int = PATH_AUTO) -> int:
    return load().w4a16_choose_split_k_ex(M, N, K, group, path)


def w4a16_choose_path(M: int, N: int, K: int, group: int = GROUP) -> int:
    return load().w4a16_choose_path(M, N, K, group)


def w4a16_set_workspace(ws: Optional[torch.Tensor]) -> None:
    """Register ``ws`` (a uint8 CUDA tensor the caller keeps alive) as the Split-K workspace."""
    if ws is None:
        _check(load().w4a16_set_workspace(None, 0), "w4a16_set_workspace")
    else:
        _check(load().w4a16_set_workspace(ws.data_ptr(), ws.numel() * ws.element_size()),
               "w4a16_set_workspace")


def w4a16_device_status() -> int:
    v = ctypes.c_int(0)
    rc = load().w4a16_device_status(ctypes.byref(v))
    if rc not in (0, -8):
        raise W4A16Error(rc, "w4a16_device_status")
    return v.value


def w4a16_selftest_wait_timeout(limit_us: int = 1000) -> None:
    """Enqueue the diagnostic kernel whose bounded wait runs out (see ``w4a16_device_status``)."""
    _check(load().w4a16_selftest_wait_timeout(int(limit_us), _stream()), "w4a16_selftest_wait_timeout")


# ------------------------------------------------------------------ operations
@dataclass
class PackedWeights:
    Wq: torch.Tensor             # uint8, opaque
    S: torch.Tensor              # uint8, opaque
    Z: Optional[torch.Tensor]    # uint8, opaque; None for a symmetric format
    N: int
    K: int
    group: int = GROUP
    flags: int = 0               # FLAG_SYMMETRIC | FLAG_BF16


def _dtype_of(flags: int):
    return torch.bfloat16 if flags & FLAG_BF16 else torch.float16


def w4a16_pack(Wq_raw: torch.Tensor, S_raw: torch.Tensor, Z_raw: Optional[torch.Tensor],
               N: int, K: int, group: int = GROUP, flags: int = 0) -> PackedWeights:
    """Raw int32/uint32 [K/8,N], 16-bit scales [K/group,N], uint8 [K/group,N] (None when symmetric)
    CUDA tensors -> packed.  ``flags == 0`` goes through ``w4a16_pack``, anything else through
    ``w4a16_pack_fmt``."""
    dev = Wq_raw.device
    sym = bool(flags & FLAG_SYMMETRIC)
    nb = (w4a16_packed_wq_bytes(N, K, group), w4a16_packed_s_bytes(N, K, group),
          0 if sym else w4a16_packed_z_bytes(N, K, group))
    if nb[0] == 0:
        raise W4A16Error(-2, "w4a16_pack")
    out = [torch.empty(b, dtype=torch.uint8, device=dev) if b else None for b in nb]
    if flags == 0:
        _check(load().w4a16_pack(_ptr(Wq_raw), _ptr(S_raw), _ptr(Z_raw), _ptr(out[0]), _ptr(out[1]),
                                 _ptr(out[2]), N, K, group, _stream()), "w4a16_pack")
    else:
        _check(load().w4a16_pack_fmt(_ptr(Wq_raw), _ptr(S_raw), None if sym else _ptr(Z_raw), _ptr(out[0]),
                                     _ptr(out[1]), _ptr(out[2]), N, K, group, flags, _stream()), "w4a16_pack_fmt")
    return PackedWeights(out[0], out[1], out[2], N, K, group, flags)


def w4a16_quantize(W16: torch.Tensor, group: int = GROUP, flags: int = 0):
    """Eq. 1 on 16-bit weights [K, N] (CUDA tensor): returns the raw (Wq int32 [K/8, N], S 16-bit [K/group, N],
    Z uint8 [K/group, N] or None when symmetric) tensors that ``w4a16_pack`` consumes."""
    K, N = W16.shape
    dev = W16.device
    Wq = torch.empty((K // 8, N), dtype=torch.int32, device=dev)
    S = torch.empty((K // group, N), dtype=_dtype_of(flags), device=dev)
    Z = None if flags & FLAG_SYMMETRIC else torch.empty((K // group, N), dtype=torch.uint8, device=dev)
    _check(load().w4a16_quantize(_ptr(W16), _ptr(Wq), _ptr(S), _ptr(Z), N, K, group, flags, _stream()),
           "w4a16_quantize")
    return Wq, S, Z


def w4a16_dequant(pw: PackedWeights, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    if out is None:
        out = torch.empty((pw.K, pw.N), dtype=_dtype_of(pw.flags), device=pw.Wq.device)
    if pw.flags == 0:
        _check(load().w4a16_dequant(_ptr(pw.Wq), _ptr(pw.S), _ptr(pw.Z), _ptr(out), pw.N, pw.K, pw.group,
                                    _stream()), "w4a16_dequant")
    else:
        _check(load().w4a16_dequant_fmt(_ptr(pw.Wq), _ptr(pw.S), _ptr(pw.Z), _ptr(out), pw.N, pw.K, pw.group,
                                        pw.flags, _stream()), "w4a16_dequant_fmt")
    return out


def w4a16_gemm(A: torch.Tensor, pw: PackedWeights, C: Optional[torch.Tensor] = None,
               split_k: int = 0, path: int = PATH_AUTO, bias: Optional[torch.Tensor] = None,
               act: int = ACT_NONE) -> torch.Tensor:
    """C[M,N] = A[M,K] . Dequant(W); A a 16-bit CUDA tensor (FP16, or BF16 for a BF16 format), row-major
    contiguous.  Plain formats go through ``w4a16_gemm_ex``; format flags, ``bias`` or ``act`` through
    ``w4a16_gemm_fmt``."""
    M = A.shape[0]
    if C is None:
        C = torch.empty((M, pw.N), dtype=_dtype_of(pw.flags), device=A.device)
    if pw.flags == 0 and bias is None and act == ACT_NONE:
        _check(load().w4a16_gemm_ex(_ptr(A), _ptr(pw.Wq), _ptr(pw.S), _ptr(pw.Z), _ptr(C), M, pw.N, pw.K,
                                    pw.group, split_k, path, _stream()), "w4a16_gemm")
    else:
        _check(load().w4a16_gemm_fmt(_ptr(A), _ptr(pw.Wq), _ptr(pw.S), _ptr(pw.Z), _ptr(bias), _ptr(C), M, pw.N,
                                     pw.K, pw.group, split_k, path, pw.flags, act, _stream()), "w4a16_gemm_fmt")
    return C


def w4a16_gemm_host(A_host: torch.Tensor, A_dev: torch.Tensor, pw: PackedWeights,
                    C_dev: torch.Tensor, C_host: torch.Tensor, split_k: int = 0,
                    stream: Optional[int] = None) -> None:
    """Host activations in, host result out; copies and GEMM on ``stream`` (a raw ``cudaStream_t`` handle,
    e.g. ``torch.cuda.Stream().cuda_stream``) or, by default, on the current stream.  A pinned ``C_host`` is
    written by the kernel itself and ``C_dev`` is then left untouched; a pageable one goes through ``C_dev``."""
    M = A_host.shape[0]
    _check(load().w4a16_gemm_host(_ptr(A_host), _ptr(A_dev), _ptr(pw.Wq), _ptr(pw.S), _ptr(pw.Z),
                                  _ptr(C_dev), _ptr(C_host), M, pw.N, pw.K, pw.group, split_k,
                                  _stream() if stream is None else stream), "w4a16_gemm_host")


def w4a16_gemm_static_ws(A: torch.Tensor, pw: PackedWeights, C: Optional[torch.Tensor] = None,
                         split_k: int = 0) -> torch.Tensor:
    """``w4a16_gemm`` for callers that may not allocate: the Split-K scratch is an array built into
    the library, nothing is registered and the library allocates nothing.  Pass ``C`` to keep this
    wrapper from allocating the output as well.  Calls that overlap on the GPU race on the shared
    array; shapes whose scratch need exceeds it raise ``W4A16Error`` (-5)."""
    M = A.shape[0]
    if C is None:
        C = torch.empty((M, pw.N), dtype=torch.float16, device=A.device)
    _check(load().w4a16_gemm_static_ws(_ptr(A), _ptr(pw.Wq), _ptr(pw.S), _ptr(pw.Z), _ptr(C), M, pw.N,
                                       pw.K, pw.group, split_k, _stream()), "w4a16_gemm_static_ws")
    return C


def ensure_workspace(nbytes: int, device="cuda") -> torch.Tensor:
    """Allocate (with torch) and register a workspace of at least ``nbytes``; returns the tensor,
    which the caller must keep alive while it is registered."""
    ws = torch.empty(max(int(nbytes), WS_HEADER_BYTES) + 256, dtype=torch.uint8, device=device)
    off = (-ws.data_ptr()) % 256
    view = ws[off:off + max(int(nbytes), WS_HEADER_BYTES)]
    w4a16_set_workspace(view)
    view._keepalive = ws  # type: ignore[attr-defined]
    return view
