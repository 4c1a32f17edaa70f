"""Helpers for the GPU parity tests: upload a seeded problem, pack it, compare with the oracle."""
import numpy as np
import torch

from paper_2601_16536_b200 import binding as B

REL_FROB_TOL = 1e-3       # || C_gpu - C_ref ||_F / || C_ref ||_F
ELEM_TOL = 2e-3           # | dC | <= ELEM_TOL * (1 + | C_ref |)


def to_dev(a: np.ndarray) -> torch.Tensor:
    if a.dtype == np.uint32:
        return torch.from_numpy(a.view(np.int32)).cuda()
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.float16)).cuda()
    return torch.from_numpy(a).cuda()


def pack_problem(d, N, K, group=128):
    return B.w4a16_pack(to_dev(d["Wq"]), to_dev(d["S"]), to_dev(d["Z"]), N, K, group)


def c_bits(C: torch.Tensor) -> np.ndarray:
    return C.cpu().numpy().view(np.uint16)


def c_f64(C: torch.Tensor) -> np.ndarray:
    return C.cpu().numpy().astype(np.float64)


def assert_close(C_gpu: np.ndarray, C_ref: np.ndarray, what=""):
    """Relative Frobenius error <= REL_FROB_TOL and every element within ELEM_TOL (1 + |C_ref|) of the FP64 oracle."""
    mask = ~np.isnan(C_ref)
    g, r = C_gpu[mask], C_ref[mask]
    assert np.all(np.isfinite(g)), what
    frob = np.linalg.norm(g - r) / max(np.linalg.norm(r), 1e-30)
    worst = np.max(np.abs(g - r) / (1.0 + np.abs(r)))
    assert frob <= REL_FROB_TOL, "%s: rel Frobenius %.3e" % (what, frob)
    assert worst <= ELEM_TOL, "%s: worst element %.3e" % (what, worst)
    return frob, worst


def ensure_ws(M, N, K, split_k, group=128):
    splits = split_k if isinstance(split_k, (tuple, list)) else (split_k,)
    need = max([B.w4a16_workspace_bytes(M, N, K, group, s) for s in splits] + [16384])
    return B.ensure_workspace(need)
