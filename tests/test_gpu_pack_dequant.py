"""GPU: w4a16_pack is a bijection and w4a16_dequant matches the oracle bit for bit
(Algorithm 1, Phase 1: Dequant(W) = s (W - z), rounded once to FP16)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2601_16536_b200 import binding as B
from paper_2601_16536_b200 import workloads as wl
from gpu_util import pack_problem, to_dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("K,N", [(128, 64), (384, 192), (1024, 320), (4096, 4096)])
def test_dequant_bit_exact(K, N):
    d = wl.draw_weights(K, N, seed=K + N)
    pw = pack_problem(d, N, K)
    got = B.w4a16_dequant(pw).cpu().numpy().view(np.uint16)
    want = oracle.dequant(d["Wq"], d["S"], d["Z"], K, N, 128)
    assert np.array_equal(got, want)


def test_dequant_bit_exact_on_extreme_scales():
    # subnormal, tiny, huge and negative scales: one rounding, subnormals kept, Inf on overflow
    K, N = 512, 128
    d = wl.draw_weights(K, N, seed=77)
    rng = np.random.default_rng(78)
    S = rng.integers(0, 0x7C00, size=d["S"].shape).astype(np.uint16)
    S[0, :16] = [0x0001, 0x0002, 0x0003, 0x03FF, 0x0400, 0x0401, 0x7BFF, 0x7800,
                 0x8001, 0x83FF, 0xFBFF, 0x3C00, 0xBC00, 0x0000, 0x8000, 0x211F]
    d["S"] = S
    pw = pack_problem(d, N, K)
    got = B.w4a16_dequant(pw).cpu().numpy().view(np.uint16)
    want = oracle.dequant(d["Wq"], d["S"], d["Z"], K, N, 128)
    # (q - z) = 0 times a negative scale: IEEE gives -0 on both sides; compare all bits
    assert np.array_equal(got, want)


def test_pack_is_a_bijection():
    # with s = 1 and z = 0 dequant returns q itself, so pack followed by dequant must give
    # back every nibble of the raw words at its (k, n)
    K, N = 640, 256
    d = wl.draw_weights(K, N, seed=5)
    d["S"] = np.full_like(d["S"], 0x3C00)
    d["Z"] = np.zeros_like(d["Z"])
    pw = pack_problem(d, N, K)
    got = B.w4a16_dequant(pw).cpu().numpy().astype(np.int32)
    want = oracle.unpack(d["Wq"], K, N).astype(np.int32)
    assert np.array_equal(got, want)
    # and the zero points / scales land on their own (group, column)
    d2 = wl.draw_weights(K, N, seed=6)
    d2["Wq"] = np.zeros_like(d2["Wq"])            # q = 0 -> w = -z * s
    pw2 = pack_problem(d2, N, K)
    got2 = B.w4a16_dequant(pw2).cpu().numpy().view(np.uint16)
    assert np.array_equal(got2, oracle.dequant(d2["Wq"], d2["S"], d2["Z"], K, N, 128))


def test_packed_buffers_have_declared_sizes():
    K, N = 256, 128
    pw = pack_problem(wl.draw_weights(K, N, seed=1), N, K)
    assert pw.Wq.numel() == K * N // 2
    assert pw.S.numel() == (K // 128) * N * 2
    assert pw.Z.numel() == (K // 128) * N // 2


def test_pack_rejects_bad_shapes():
    x = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.W4A16Error):
        B.w4a16_pack(x, x, x, 100, 128)
