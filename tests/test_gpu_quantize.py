"""GPU: the quantizer of Eq. 1 through the C ABI, bit for bit against the oracle (codes, scales and zero
points are integers / bit patterns decided in binary32 on both sides), and the whole chain
quantize -> pack -> GEMM against the oracle's product of the weights it quantized."""
import numpy as np
import pytest
import torch

import oracle
from paper_2601_16536_b200 import binding as B
from paper_2601_16536_b200 import workloads as wl
from gpu_util import assert_close, ensure_ws

pytestmark = pytest.mark.gpu


def _weights(K, N, seed, bf16):
    r = np.random.Generator(np.random.PCG64([seed, 9]))
    x = (r.standard_normal((K, N)) * 0.04).astype(np.float32)
    x[::97, ::5] *= 6.0                                   # a few outliers per group
    x[128:256, 3] = 0.0                                   # a group of zeros
    x[256:384, 4] = 0.0123                                # a constant group
    return wl._bits16(x, bf16)


@pytest.mark.parametrize("group", [32, 64, 128])
@pytest.mark.parametrize("symmetric", [False, True])
@pytest.mark.parametrize("bf16", [False, True])
def test_quantize_is_bit_exact(group, symmetric, bf16):
    K, N = 512, 192
    bits = _weights(K, N, group + symmetric, bf16)
    flags = (B.FLAG_SYMMETRIC if symmetric else 0) | (B.FLAG_BF16 if bf16 else 0)
    W = torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16 if bf16 else torch.float16)
    Wq, S, Z = B.w4a16_quantize(W, group, flags)
    torch.cuda.synchronize()
    wq, s, z = oracle.quantize(bits, K, N, group, symmetric=symmetric, bf16=bf16)
    assert np.array_equal(Wq.cpu().numpy().view(np.uint32), wq)
    assert np.array_equal(S.view(torch.int16).cpu().numpy().view(np.uint16), s)
    if symmetric:
        assert Z is None and np.all(z == 8)
    else:
        assert np.array_equal(Z.cpu().numpy(), z)


@pytest.mark.parametrize("M,symmetric", [(4, False), (4, True), (48, False)])
def test_quantize_pack_gemm_chain(M, symmetric):
    K, N, group = 2048, 512, 128
    bits = _weights(K, N, 5, False)
    flags = B.FLAG_SYMMETRIC if symmetric else 0
    W = torch.from_numpy(bits.view(np.float16)).cuda()
    Wq, S, Z = B.w4a16_quantize(W, group, flags)
    pw = B.w4a16_pack(Wq, S, Z, N, K, group, flags)
    A_bits = wl.draw_activations(M, K, 17)
    ws = ensure_ws(M, N, K, 0)
    C = B.w4a16_gemm(torch.from_numpy(A_bits.view(np.float16)).cuda(), pw)
    torch.cuda.synchronize()
    assert B.w4a16_device_status() == 0
    wq, s, z = oracle.quantize(bits, K, N, group, symmetric=symmetric)
    ref = oracle.gemm(A_bits, wq, s, z, M, N, K, group)
    assert_close(C.cpu().numpy().astype(np.float64), ref, "chain M%d sym%d" % (M, symmetric))
    # and the quantized product stays close to the product with the original FP16 weights (4-bit error)
    full = A_bits.view(np.float16).astype(np.float64) @ bits.view(np.float16).astype(np.float64)
    assert np.linalg.norm(ref - full) / np.linalg.norm(full) < 0.2
    del ws
