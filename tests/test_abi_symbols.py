"""The C-ABI library loads, exports every symbol include/w4a16.h declares, and validates
arguments on the host before touching a device (no compute calls here)."""
import ctypes
import os
import re

import pytest

from paper_2601_16536_b200 import binding as B
from paper_2601_16536_b200 import build as libbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    libbuild.build_library()
    return B.load()


def _declared():
    text = open(os.path.join(ROOT, "include", "w4a16.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(w4a16_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert len(names) >= 12
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(B.EXPORTS)


def test_packed_sizes_hold_exactly_the_raw_information(lib):
    for N, K in [(64, 128), (4096, 4096), (4096, 11008), (8192, 28672), (22016, 4096)]:
        assert lib.w4a16_packed_wq_bytes(N, K, 128) == K * N // 2
        assert lib.w4a16_packed_s_bytes(N, K, 128) == (K // 128) * N * 2
        assert lib.w4a16_packed_z_bytes(N, K, 128) == (K // 128) * N // 2
    # unsupported shapes report size 0
    assert lib.w4a16_packed_wq_bytes(100, 4096, 128) == 0
    assert lib.w4a16_packed_wq_bytes(4096, 4000, 128) == 0
    assert lib.w4a16_packed_wq_bytes(4096, 4096, 48) == 0
    # smaller quantization groups: the same nibbles, proportionally more scales and zero points
    for group in (32, 64):
        assert lib.w4a16_packed_wq_bytes(4096, 4096, group) == 4096 * 4096 // 2
        assert lib.w4a16_packed_s_bytes(4096, 4096, group) == (4096 // group) * 4096 * 2
        assert lib.w4a16_packed_z_bytes(4096, 4096, group) == (4096 // group) * 4096 // 2


def test_choose_split_k_is_always_acceptable(lib):
    for M in (1, 2, 4, 8, 16, 32, 64, 256, 1024, 4096):
        for N, K in [(4096, 4096), (4096, 11008), (8192, 28672), (12288, 4096), (22016, 4096),
                     (8192, 8192), (64, 128), (64, 256)]:
            s = lib.w4a16_choose_split_k(M, N, K, 128)
            assert 1 <= s <= K // 128
            for path in (1, 2, 3):
                s = lib.w4a16_choose_split_k_ex(M, N, K, 128, path)
                assert 1 <= s <= K // 128
            # automatic scheduling shares column tiles between CTAs, so it needs partial-tile slots
            assert lib.w4a16_workspace_bytes(M, N, K, 128, 0) >= 16384
            assert lib.w4a16_workspace_bytes(M, N, K, 128, 1) == 0
    assert lib.w4a16_workspace_bytes(4, 4096, 4096, 128, 1) == 0
    assert lib.w4a16_workspace_bytes(4, 4096, 4096, 128, 4) >= 4 * 4 * 4096 * 4


def test_schedule_queries_are_consistent_on_a_grid_of_shapes(lib):
    """Host logic over 675 (M, N, K, group) combinations, none of them tuned for: the path is one of the two
    GEMM kernels, the reported split is one w4a16_gemm accepts (1 .. K/128 for every group size), a split of
    1 needs no workspace, any other split needs at least the ticket header, and the size is bounded by the
    partial tiles the schedule can produce (two per CTA slot of a 148-SM device, per batch chunk)."""
    header = 16384 + 131072
    n = 0
    for group in (32, 64, 128):
        for M in (1, 3, 8, 9, 16, 17, 64, 300, 4096):
            for N in (64, 1536, 4096, 4608, 22016):
                for K in (128, 1024, 4096, 11008, 28672):
                    n += 1
                    blocks = K // 128
                    assert lib.w4a16_choose_path(M, N, K, group) in (2, 3)
                    s = lib.w4a16_choose_split_k(M, N, K, group)
                    assert 1 <= s <= blocks, (M, N, K, group, s)
                    for path in (1, 2, 3):
                        assert 1 <= lib.w4a16_choose_split_k_ex(M, N, K, group, path) <= blocks
                    assert lib.w4a16_workspace_bytes(M, N, K, group, 1) == 0
                    assert lib.w4a16_workspace_bytes(M, N, K, group, blocks + 1) == 0      # not a valid split
                    for split in {0, s, min(2, blocks), blocks}:
                        if split == 1:
                            continue
                        need = lib.w4a16_workspace_bytes(M, N, K, group, split)
                        assert need == 0 or need >= header
                        # plain path: split x M x N floats; warp-MMA path: two 16 x 64 tiles per chunk and batch
                        # chunk; tcgen05 path: two MT x 128 tiles per chunk
                        sp = split if split else max(s, 1)
                        bound = header + 256 + max(4 * sp * M * N,
                                                   2 * max(296, (N // 64) * sp) * ((M + 15) // 16) * 16 * 64 * 4,
                                                   2 * max(148, ((M + 15) // 16) * ((N + 127) // 128) * sp) * 256 * 128 * 4)
                        assert need <= bound, (M, N, K, group, split, need, bound)
    assert n == 675


def test_path_and_schedule_rules_at_the_benchmark_shapes(lib):
    """Host logic only (148 SMs assumed without a device, which is also what a B200 reports): the
    path and the split the library reports for a shape are the ones it runs (w4a16_gemm asks the same
    functions).  Values are the measured optima recorded beside the rules in the sources."""
    DECODE, TILE = 2, 3
    path = lambda M, N, K: lib.w4a16_choose_path(M, N, K, 128)
    split = lambda M, N, K: lib.w4a16_choose_split_k(M, N, K, 128)
    # up to 16 rows (one pass of the warp-MMA kernel over the weights): always that kernel
    for N, K in [(4096, 4096), (4096, 11008), (8192, 28672), (22016, 4096), (1536, 6144), (12288, 4096)]:
        for M in (1, 4, 8, 9, 16):
            assert path(M, N, K) == DECODE
    assert split(16, 4096, 11008) == 4
    # above 16 rows: tcgen05
    for M in (17, 32, 64, 256, 4096):
        assert path(M, 4096, 11008) == TILE
    # slices per tile of the warp-MMA kernel: four (one cluster per tile) at config 2, whole tiles
    # for the wide gate/up layer, at most six per cluster for narrow matrices
    assert split(1, 4096, 11008) == 4
    assert split(1, 4096, 4096) == 4
    assert split(1, 22016, 4096) == 1
    assert split(1, 12288, 4096) == 1
    assert split(1, 1536, 6144) == 6
    assert split(1, 2048, 8192) == 6
    # wide batch tiles: whole tiles at M = 4096 (no partial tiles at all)
    assert split(4096, 8192, 8192) == 1
    # unsupported shapes are refused, not guessed
    assert lib.w4a16_choose_path(1, 100, 4096, 128) < 0


def test_argument_errors_are_reported_before_any_device_work(lib):
    buf = (ctypes.c_uint8 * 4096)()
    p = ctypes.addressof(buf)
    p = (p + 15) // 16 * 16
    assert lib.w4a16_gemm(None, p, p, p, p, 1, 64, 128, 128, 1, None) == -1
    assert lib.w4a16_gemm(p, p, p, p, None, 1, 64, 128, 128, 1, None) == -1
    assert lib.w4a16_gemm(p, p, p, p, p, 1, 64, 128, 48, 1, None) == -2      # group
    assert lib.w4a16_gemm(p, p, p, p, p, 1, 60, 128, 128, 1, None) == -2     # N % 64
    assert lib.w4a16_gemm(p, p, p, p, p, 1, 64, 100, 128, 1, None) == -2     # K % 128
    assert lib.w4a16_gemm(p, p, p, p, p, 0, 64, 128, 128, 1, None) == -2     # M
    assert lib.w4a16_gemm(p + 2, p, p, p, p, 1, 64, 128, 128, 1, None) == -3  # alignment
    assert lib.w4a16_gemm(p, p, p, p, p, 1, 64, 128, 128, 2, None) == -4     # split_k > K/group
    assert lib.w4a16_gemm(p, p, p, p, p, 1, 64, 128, 128, -1, None) == -4
    assert lib.w4a16_gemm_ex(p, p, p, p, p, 1, 64, 128, 128, 1, 9, None) == -9
    assert lib.w4a16_pack(None, p, p, p, p, p, 64, 128, 128, None) == -1
    assert lib.w4a16_pack(p, p, p, p, p, p, 64, 128, 16, None) == -2
    assert lib.w4a16_pack(p, p, None, p, p, p, 64, 128, 128, None) == -1      # the plain entry points need Z
    assert lib.w4a16_gemm(p, p, p, None, p, 1, 64, 128, 128, 1, None) == -1
    assert lib.w4a16_pack_fmt(p, p, None, p, p, None, 64, 128, 128, 0, None) == -1   # asymmetric: Z required
    assert lib.w4a16_pack_fmt(p, p, None, p, p, None, 64, 128, 128, 8, None) == -2   # unknown flag
    assert lib.w4a16_gemm_fmt(p, p, p, None, None, p, 1, 64, 128, 128, 1, 0, 0, 0, None) == -1
    assert lib.w4a16_gemm_fmt(p, p, p, p, None, p, 1, 64, 128, 128, 1, 0, 0, 7, None) == -2   # unknown activation
    assert lib.w4a16_gemm_fmt(p, p, p, p, p + 1, p, 1, 64, 128, 128, 1, 0, 0, 0, None) == -3  # odd bias address
    assert lib.w4a16_dequant_fmt(p, p, None, p, 64, 128, 128, 0, None) == -1
    assert lib.w4a16_dequant(p, p, p, None, 64, 128, 128, None) == -1
    assert lib.w4a16_dequant(p, p, p, p + 4, 64, 128, 128, None) == -3
    assert lib.w4a16_gemm_host(None, p, p, p, p, p, p, 1, 64, 128, 128, 1, None) == -1
    assert lib.w4a16_device_status(None) == -1
    for code in range(-9, 1):
        assert len(B.strerror(code)) > 1


def test_binding_refuses_to_run_without_the_library(monkeypatch, tmp_path):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        B.load()
