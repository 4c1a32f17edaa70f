// pack (offline reorder), standalone dequant, the plain FP32-FMA GEMM and the Split-K
// reduce kernel.
#pragma once

#include "common.cuh"

namespace w4a16 {

// ------------------------------------------------------------------ pack
// One thread per packed word.  Pure bit moves (Section 2.2 storage packing).
__global__ void pack_wq_kernel(const uint32_t* __restrict__ raw, uint32_t* __restrict__ out, int N, int G,
                               size_t total_words) {
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total_words) return;
    int j = (int)(idx & 3);
    int lane = (int)((idx >> 2) & 31);
    int r = (int)((idx >> 7) & 3);
    int c = (int)((idx >> 9) & 1);
    size_t blk = idx >> 10;
    int t = (int)(blk / G), g = (int)(blk % G);
    int tig = lane & 3, gq = lane >> 2;
    int n_lo = t * kTileN + r * 16 + gq;
    int k0 = g * kGroup + c * 64 + tig * 16 + j * 4;
    int sh = (k0 & 7) * 4;  // 0 or 16: the four k sit in one half of a raw word
    uint32_t a = (raw[(size_t)(k0 >> 3) * N + n_lo] >> sh) & 0xFFFFu;
    uint32_t b = (raw[(size_t)(k0 >> 3) * N + n_lo + 8] >> sh) & 0xFFFFu;
    uint32_t a0 = a & 15u, a1 = (a >> 4) & 15u, a2 = (a >> 8) & 15u, a3 = (a >> 12) & 15u;
    uint32_t b0 = b & 15u, b1 = (b >> 4) & 15u, b2 = (b >> 8) & 15u, b3 = (b >> 12) & 15u;
    out[idx] = a0 | (b0 << 4) | (a2 << 8) | (b2 << 12) | (a1 << 16) | (b1 << 20) | (a3 << 24) | (b3 << 28);
}

__global__ void pack_s_kernel(const uint16_t* __restrict__ raw, uint16_t* __restrict__ out, int N, int G,
                              size_t total) {
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total) return;
    int e = (int)(idx & 63);
    size_t blk = idx >> 6;
    int t = (int)(blk / G), g = (int)(blk % G);
    int gq = e >> 3, r = (e >> 1) & 3, h = e & 1;
    out[idx] = raw[(size_t)g * N + t * kTileN + r * 16 + gq + 8 * h];
}

__global__ void pack_z_kernel(const uint8_t* __restrict__ raw, uint32_t* __restrict__ out, int N, int G,
                              size_t total_words) {
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total_words) return;
    int gq = (int)(idx & 7);
    size_t blk = idx >> 3;
    int t = (int)(blk / G), g = (int)(blk % G);
    uint32_t w = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        int r = i >> 1, h = i & 1;
        w |= (uint32_t)(raw[(size_t)g * N + t * kTileN + r * 16 + gq + 8 * h] & 15u) << (4 * i);
    }
    out[idx] = w;
}

// ------------------------------------------------------------------ dequant
// Algorithm 1, Phase 1 as a standalone kernel: one thread per packed word, eight FP16
// results w16 = fp16_rn((q - z) * s): (q - z) is formed exactly in FP16 and multiplied by s
// with one FP16 multiply (round-to-nearest-even, subnormals kept).
__global__ void dequant_kernel(const uint32_t* __restrict__ Wq, const __half* __restrict__ S,
                               const uint32_t* __restrict__ Z, __half* __restrict__ W16, int N, int G,
                               size_t total_words) {
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total_words) return;
    int j = (int)(idx & 3);
    int lane = (int)((idx >> 2) & 31);
    int r = (int)((idx >> 7) & 3);
    int c = (int)((idx >> 9) & 1);
    size_t blk = idx >> 10;
    int t = (int)(blk / G), g = (int)(blk % G);
    int tig = lane & 3, gq = lane >> 2;
    int n_lo = t * kTileN + r * 16 + gq;
    int k0 = g * kGroup + c * 64 + tig * 16 + j * 4;

    uint32_t zw = Z[blk * kZBlockWords + gq];
    __half2 zlo = u32_as_h2(zmagic_lo((zw >> (8 * r)) & 15u));
    __half2 zhi = u32_as_h2(zmagic_hi((zw >> (8 * r + 4)) & 15u));
    __half s_lo = S[blk * kSBlockHalves + gq * 8 + r * 2];
    __half s_hi = S[blk * kSBlockHalves + gq * 8 + r * 2 + 1];

    const Frag4 f = dequant_word(Wq[idx], zlo, zhi, __half2half2(s_lo), __half2half2(s_hi));
    const __half2 wa = f.lo_a, wb = f.lo_b, wc = f.hi_a, wd = f.hi_b;
    __half* p = W16 + (size_t)k0 * N + n_lo;
    p[0] = __low2half(wa);
    p[(size_t)N] = __high2half(wa);
    p[(size_t)2 * N] = __low2half(wb);
    p[(size_t)3 * N] = __high2half(wb);
    p[8] = __low2half(wc);
    p[(size_t)N + 8] = __high2half(wc);
    p[(size_t)2 * N + 8] = __low2half(wd);
    p[(size_t)3 * N + 8] = __high2half(wd);
}

// ------------------------------------------------------------------ plain GEMM
// Correct-first kernel: one thread per output column of a 64-column tile, kSimpleMB batch
// rows per thread, FP32 FMA in ascending k over this CTA's K-slice.  Grid: (N/64,
// ceil(M/kSimpleMB), split_k).  With split_k == 1 it writes FP16 C, else FP32 partials
// ws[split][M][N] (Algorithm 1, Phase 2) for splitk_reduce_kernel.
constexpr int kSimpleMB = 4;

__device__ __forceinline__ void slice_of(int G, int split_k, int sp, int& g0, int& ng) {
    int base = G / split_k, rem = G % split_k;
    g0 = sp * base + min(sp, rem);
    ng = base + (sp < rem ? 1 : 0);
}

__global__ void __launch_bounds__(64)
gemm_simple_kernel(const __half* __restrict__ A, const uint32_t* __restrict__ Wq, const __half* __restrict__ S,
                   const uint32_t* __restrict__ Z, __half* __restrict__ C, float* __restrict__ ws, int M, int N,
                   int K, int G, int split_k) {
    int t = blockIdx.x, m0 = blockIdx.y * kSimpleMB, sp = blockIdx.z;
    int e = threadIdx.x;  // row inside the tile
    int r = e >> 4, gq = e & 7, h = (e >> 3) & 1;
    int g0, ng;
    slice_of(G, split_k, sp, g0, ng);

    float acc[kSimpleMB];
#pragma unroll
    for (int i = 0; i < kSimpleMB; ++i) acc[i] = 0.f;

    for (int g = g0; g < g0 + ng; ++g) {
        size_t blk = (size_t)t * G + g;
        int z = (int)((Z[blk * kZBlockWords + gq] >> (4 * (r * 2 + h))) & 15u);
        float s = __half2float(S[blk * kSBlockHalves + gq * 8 + r * 2 + h]);
        const uint32_t* wb = Wq + blk * kBlockWords;
        for (int c = 0; c < 2; ++c)
            for (int tig = 0; tig < 4; ++tig)
                for (int j = 0; j < 4; ++j) {
                    uint32_t w = wb[((c * 4 + r) * 32 + gq * 4 + tig) * 4 + j] >> (4 * h);
                    int k0 = g * kGroup + c * 64 + tig * 16 + j * 4;
                    // nibbles (after the shift by 4h): 0 -> k0, 4 -> k0+1, 2 -> k0+2, 6 -> k0+3
                    int q[4] = {(int)(w & 15u), (int)((w >> 16) & 15u), (int)((w >> 8) & 15u),
                                (int)((w >> 24) & 15u)};
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        float w16 = __half2float(__float2half_rn((float)(q[i] - z) * s));
#pragma unroll
                        for (int mm = 0; mm < kSimpleMB; ++mm) {
                            if (m0 + mm < M)
                                acc[mm] = fmaf(__half2float(A[(size_t)(m0 + mm) * K + k0 + i]), w16, acc[mm]);
                        }
                    }
                }
    }
    int n = t * kTileN + r * 16 + gq + 8 * h;
#pragma unroll
    for (int mm = 0; mm < kSimpleMB; ++mm) {
        if (m0 + mm < M) {
            if (split_k == 1)
                C[(size_t)(m0 + mm) * N + n] = __float2half_rn(acc[mm]);
            else
                ws[((size_t)sp * M + m0 + mm) * N + n] = acc[mm];
        }
    }
}

// Algorithm 1, Phase 3: C = fp16_rn(sum_{i<S} C_i), ascending i, FP32.
__global__ void splitk_reduce_kernel(const float* __restrict__ ws, __half* __restrict__ C, size_t MN,
                                     int split_k) {
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= MN) return;
    float acc = ws[i];
    for (int s = 1; s < split_k; ++s) acc += ws[(size_t)s * MN + i];
    C[i] = __float2half_rn(acc);
}

}  // namespace w4a16
