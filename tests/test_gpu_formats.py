"""GPU parity of the format variants through the C ABI (w4a16_pack_fmt / w4a16_dequant_fmt /
w4a16_gemm_fmt): quantization groups of 32 and 64 along K, the symmetric case of Eq. 1 (zero point 8,
no Z buffer), BF16 instead of FP16 (Section 1 names both as the dequantization target), and the fused
bias / activation step.  Dequantization is compared bit for bit, products within the GEMM tolerances,
exactly representable inputs bit for bit on every path and split."""
import numpy as np
import pytest
import torch

import oracle
from paper_2601_16536_b200 import binding as B
from paper_2601_16536_b200 import workloads as wl
from gpu_util import assert_close, ensure_ws, to_dev

pytestmark = pytest.mark.gpu

PATHS = {"simple": B.PATH_SIMPLE, "decode": B.PATH_DECODE, "tile": B.PATH_TILE}


def _flags(symmetric, bf16=False):
    return (B.FLAG_SYMMETRIC if symmetric else 0) | (B.FLAG_BF16 if bf16 else 0)


def _dev16(bits, bf16=False):
    t = torch.from_numpy(bits.view(np.int16)).cuda()
    return t.view(torch.bfloat16 if bf16 else torch.float16)


def _pack(d, N, K, group, symmetric, bf16=False):
    return B.w4a16_pack(to_dev(d["Wq"]), _dev16(d["S"], bf16), None if symmetric else to_dev(d["Z"]), N, K, group,
                        _flags(symmetric, bf16))


def _bits(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def _f64(t):
    return t.to(torch.float32).cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("group", [32, 64, 128])
@pytest.mark.parametrize("symmetric", [False, True])
def test_dequant_is_bit_exact(group, symmetric):
    K, N = 640, 192      # five k-blocks, three column tiles
    d = wl.draw_weights(K, N, seed=800 + group, group=group, symmetric=symmetric)
    # scales over the whole FP16 range, subnormal and huge ones among them
    r = np.random.Generator(np.random.PCG64(group))
    d["S"] = r.integers(0, 0x7C00, size=d["S"].shape, dtype=np.uint64).astype(np.uint16)
    pw = _pack(d, N, K, group, symmetric)
    assert (pw.Z is None) == symmetric
    got = _bits(B.w4a16_dequant(pw))
    want = oracle.dequant(d["Wq"], d["S"], d["Z"], K, N, group)
    assert np.array_equal(got, want)


SHAPES = [(1, 640, 192), (5, 1152, 128), (16, 896, 256), (40, 768, 128)]


@pytest.mark.parametrize("path", list(PATHS))
@pytest.mark.parametrize("group,symmetric", [(32, False), (64, False), (128, True), (32, True), (64, True)])
@pytest.mark.parametrize("M,K,N", SHAPES)
def test_gemm_matches_oracle(path, group, symmetric, M, K, N):
    d = wl.make_problem(M, K, N, seed=M + K + group, group=group, symmetric=symmetric)
    pw = _pack(d, N, K, group, symmetric)
    ws = ensure_ws(M, N, K, (0, 1, 2, 3))
    ref = oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, group)
    for split_k in (0, 1, 3):
        C = B.w4a16_gemm(_dev16(d["A"]), pw, split_k=split_k, path=PATHS[path])
        torch.cuda.synchronize()
        assert B.w4a16_device_status() == 0
        assert_close(_f64(C), ref, "%s g%d sym%d M%d split %d" % (path, group, symmetric, M, split_k))
    del ws


@pytest.mark.parametrize("path", list(PATHS))
@pytest.mark.parametrize("group,symmetric", [(32, False), (64, True), (128, True)])
def test_exact_inputs_are_bit_equal(path, group, symmetric):
    M, K, N = 7, 1152, 128
    d = wl.make_exact_problem(M, K, N, seed=31 + group, group=group, symmetric=symmetric)
    pw = _pack(d, N, K, group, symmetric)
    want = oracle.gemm_int(d["A_int"], d["Wq"], d["E"], d["Z"], M, N, K, group)
    ws = ensure_ws(M, N, K, (0, 1, 2, 4, 9))
    for split_k in (0, 1, 2, 4, 9):
        C = B.w4a16_gemm(_dev16(d["A"]), pw, split_k=split_k, path=PATHS[path])
        torch.cuda.synchronize()
        assert np.array_equal(_bits(C), want), "split_k=%d" % split_k
    del ws


@pytest.mark.parametrize("group,symmetric", [(32, False), (64, False), (128, True)])
def test_full_size_decode_shape_whole_output(group, symmetric):
    # the benchmark's decode shape with the format variants, automatic path and split, whole C
    M, K, N = 8, 11008, 4096
    d = wl.make_problem(M, K, N, seed=group, group=group, symmetric=symmetric)
    pw = _pack(d, N, K, group, symmetric)
    ws = ensure_ws(M, N, K, 0)
    C = B.w4a16_gemm(_dev16(d["A"]), pw)
    torch.cuda.synchronize()
    assert B.w4a16_device_status() == 0
    assert_close(_f64(C), oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, group), "g%d sym%d" % (group, symmetric))
    del ws


@pytest.mark.parametrize("path,M", [("simple", 3), ("decode", 6), ("decode", 16), ("tile", 24), ("tile", 200)])
@pytest.mark.parametrize("act", ["none", "relu", "silu"])
def test_bias_and_activation_are_applied_before_the_final_rounding(path, M, act):
    K, N = 1152, 256
    d = wl.make_problem(M, K, N, seed=M * 7 + len(act))
    pw = _pack(d, N, K, 128, False)
    r = np.random.Generator(np.random.PCG64(M))
    bias_bits = r.standard_normal(N).astype(np.float16).view(np.uint16)
    bias = bias_bits.view(np.float16).astype(np.float64)
    ws = ensure_ws(M, N, K, (0, 1, 3))
    ref = oracle.epilogue(oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, 128), bias, act)
    code = {"none": B.ACT_NONE, "relu": B.ACT_RELU, "silu": B.ACT_SILU}[act]
    for split_k in (0, 1, 3):
        C = B.w4a16_gemm(_dev16(d["A"]), pw, split_k=split_k, path=PATHS[path], bias=_dev16(bias_bits), act=code)
        torch.cuda.synchronize()
        assert B.w4a16_device_status() == 0
        assert_close(_f64(C), ref, "%s M%d %s split %d" % (path, M, act, split_k))
        if act == "relu":
            assert np.all(_f64(C) >= 0)
    del ws


@pytest.mark.parametrize("bf16", [False, True])
def test_bias_and_activation_after_the_second_kernels_sum(bf16):
    """256-row tiles in K slices: the partial tiles are summed by a kernel of their own, which then also adds
    the bias and applies the activation before the one rounding."""
    M, K, N = 150, 1024, 1536
    d = wl.make_problem(M, K, N, seed=911, bf16=bf16)
    pw = _pack(d, N, K, 128, False, bf16=bf16)
    r = np.random.Generator(np.random.PCG64(5))
    bias32 = r.standard_normal(N).astype(np.float32)
    if bf16:
        bias_bits = (bias32.view(np.uint32) >> 16).astype(np.uint16)
        bias = (bias_bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    else:
        bias_bits = bias32.astype(np.float16).view(np.uint16)
        bias = bias_bits.view(np.float16).astype(np.float64)
    ws = ensure_ws(M, N, K, (0, 4))
    ref = oracle.epilogue(oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, 128, bf16=bf16), bias, "silu")
    for split_k in (0, 4):
        C = B.w4a16_gemm(_dev16(d["A"], bf16), pw, split_k=split_k, path=B.PATH_TILE, bias=_dev16(bias_bits, bf16), act=B.ACT_SILU)
        torch.cuda.synchronize()
        assert B.w4a16_device_status() == 0
        if bf16:
            _assert_close_bf16(_f64(C), ref, "bf16 split %d" % split_k)
        else:
            assert_close(_f64(C), ref, "f16 split %d" % split_k)
    del ws


# ------------------------------------------------------------------ BF16
@pytest.mark.parametrize("group,symmetric", [(128, False), (64, False), (32, True)])
def test_bf16_dequant_is_bit_exact(group, symmetric):
    K, N = 512, 128
    d = wl.draw_weights(K, N, seed=900 + group, group=group, symmetric=symmetric, bf16=True)
    r = np.random.Generator(np.random.PCG64(group + 1))
    d["S"] = r.integers(0, 0x7F80, size=d["S"].shape, dtype=np.uint64).astype(np.uint16)   # the whole BF16 range
    pw = _pack(d, N, K, group, symmetric, bf16=True)
    got = _bits(B.w4a16_dequant(pw))
    want = oracle.dequant(d["Wq"], d["S"], d["Z"], K, N, group, bf16=True)
    assert np.array_equal(got, want)


# BF16 keeps 8 significant bits: the rounding of C itself is 2^-9 relative, so the tolerances of the FP16
# product (1e-3 Frobenius, 2e-3 per element) are widened by the ratio of the two formats' precision, 2^3
BF16_FROB, BF16_ELEM = 8e-3, 1.6e-2


def _assert_close_bf16(C, ref, what):
    frob = np.linalg.norm(C - ref) / max(np.linalg.norm(ref), 1e-30)
    worst = np.max(np.abs(C - ref) / (1.0 + np.abs(ref)))
    assert np.all(np.isfinite(C)), what
    assert frob <= BF16_FROB, "%s: rel Frobenius %.3e" % (what, frob)
    assert worst <= BF16_ELEM, "%s: worst element %.3e" % (what, worst)


@pytest.mark.parametrize("path", list(PATHS))
@pytest.mark.parametrize("group,symmetric", [(128, False), (64, True), (32, False)])
@pytest.mark.parametrize("M,K,N", [(1, 640, 192), (12, 1152, 128), (40, 768, 256)])
def test_bf16_gemm_matches_oracle(path, group, symmetric, M, K, N):
    d = wl.make_problem(M, K, N, seed=M + K + group, group=group, symmetric=symmetric, bf16=True)
    pw = _pack(d, N, K, group, symmetric, bf16=True)
    ws = ensure_ws(M, N, K, (0, 1, 3))
    ref = oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, group, bf16=True)
    for split_k in (0, 1, 3):
        C = B.w4a16_gemm(_dev16(d["A"], True), pw, split_k=split_k, path=PATHS[path])
        torch.cuda.synchronize()
        assert B.w4a16_device_status() == 0
        assert C.dtype == torch.bfloat16
        _assert_close_bf16(_f64(C), ref, "bf16 %s g%d sym%d M%d split %d" % (path, group, symmetric, M, split_k))
    del ws


@pytest.mark.parametrize("path", list(PATHS))
def test_bf16_exact_inputs_are_bit_equal(path):
    M, K, N = 6, 1152, 128
    d = wl.make_exact_problem(M, K, N, seed=77, bf16=True)
    pw = _pack(d, N, K, 128, False, bf16=True)
    want = oracle.gemm_int(d["A_int"], d["Wq"], d["E"], d["Z"], M, N, K, 128, bf16=True)
    ws = ensure_ws(M, N, K, (0, 1, 2, 4, 9))
    for split_k in (0, 1, 2, 4, 9):
        C = B.w4a16_gemm(_dev16(d["A"], True), pw, split_k=split_k, path=PATHS[path])
        torch.cuda.synchronize()
        assert np.array_equal(_bits(C), want), "split_k=%d" % split_k
    del ws


@pytest.mark.parametrize("M", [4, 16, 128])
def test_bf16_full_size_layer_whole_output(M):
    K, N = 4096, 4096
    d = wl.make_problem(M, K, N, seed=300 + M, bf16=True)
    pw = _pack(d, N, K, 128, False, bf16=True)
    ws = ensure_ws(M, N, K, 0)
    C = B.w4a16_gemm(_dev16(d["A"], True), pw)
    torch.cuda.synchronize()
    assert B.w4a16_device_status() == 0
    _assert_close_bf16(_f64(C), oracle.gemm(d["A"], d["Wq"], d["S"], d["Z"], M, N, K, 128, bf16=True), "bf16 M%d" % M)
    del ws
