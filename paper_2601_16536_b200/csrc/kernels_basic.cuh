// pack (offline reorder), standalone dequant, the plain FP32-FMA GEMM and the Split-K
// reduce kernel.
#pragma once

#include "common.cuh"

namespace w4a16 {

// ------------------------------------------------------------------ pack
// Decode a packed word's position: idx -> block, column inside the tile, first k inside the group.
__device__ __forceinline__ void word_position(size_t idx, size_t& blk, int& col, int& kw) {
    const int within = (int)(idx & 1023);
    blk = idx >> 10;
    const int c = within >> 9, rb = (within >> 6) & 7, i = (within >> 5) & 1, slot = (within >> 2) & 7;
    col = rb * 8 + ((slot - 4 * i) & 7);
    kw = c * 8 + i * 4 + (within & 3);
}

// One thread per packed word.  Pure bit moves (Section 2.2 storage packing): the word's eight k
// are one raw word of the same column; only the nibble order inside the word changes.
__global__ void pack_wq_kernel(const uint32_t* __restrict__ raw, uint32_t* __restrict__ out, int N, int G,
                               size_t total_words) {
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total_words) return;
    size_t blk;
    int col, kw;
    word_position(idx, blk, col, kw);
    const int t = (int)(blk / G), g = (int)(blk % G);
    const uint32_t r = raw[(size_t)(g * (kGroup / 8) + kw) * N + (size_t)t * kTileN + col];
    uint32_t w = 0;
#pragma unroll
    for (int p = 0; p < 8; ++p) {
        const int off = 2 * (p & 3) + (p >> 2);  // k offset held by nibble p
        w |= ((r >> (4 * off)) & 15u) << (4 * p);
    }
    out[idx] = w;
}

__global__ void pack_s_kernel(const uint16_t* __restrict__ raw, uint16_t* __restrict__ out, int N, int G,
                              size_t total) {
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total) return;
    const int col = (int)(idx & 63);
    const size_t blk = idx >> 6;
    const int t = (int)(blk / G), g = (int)(blk % G);
    out[idx] = raw[(size_t)g * N + (size_t)t * kTileN + col];
}

__global__ void pack_z_kernel(const uint8_t* __restrict__ raw, uint32_t* __restrict__ out, int N, int G,
                              size_t total_words) {
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total_words) return;
    const int rb = (int)(idx & 7);
    const size_t blk = idx >> 3;
    const int t = (int)(blk / G), g = (int)(blk % G);
    uint32_t w = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i)
        w |= (uint32_t)(raw[(size_t)g * N + (size_t)t * kTileN + rb * 8 + i] & 15u) << (4 * i);
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
    size_t blk;
    int col, kw;
    word_position(idx, blk, col, kw);
    const int t = (int)(blk / G), g = (int)(blk % G);
    const uint32_t z = (Z[blk * kZBlockWords + (col >> 3)] >> (4 * (col & 7))) & 15u;
    const __half s = S[blk * kSBlockHalves + col];
    const Half8 f = dequant_word(Wq[idx], u32_as_h2(zmagic_lo(z)), u32_as_h2(zmagic_hi(z)), __half2half2(s));
    __half* p = W16 + (size_t)(g * kGroup + kw * 8) * N + (size_t)t * kTileN + col;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        p[(size_t)(2 * j) * N] = __low2half(f.h[j]);
        p[(size_t)(2 * j + 1) * N] = __high2half(f.h[j]);
    }
}

// ------------------------------------------------------------------ plain GEMM
// Correct-first kernel: one thread per output column of a 64-column tile, kSimpleMB batch
// rows per thread, FP32 FMA over this CTA's K-slice.  Grid: (N/64,
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
    const int t = blockIdx.x, m0 = blockIdx.y * kSimpleMB, sp = blockIdx.z;
    const int col = threadIdx.x;  // column inside the tile
    int g0, ng;
    slice_of(G, split_k, sp, g0, ng);

    float acc[kSimpleMB];
#pragma unroll
    for (int i = 0; i < kSimpleMB; ++i) acc[i] = 0.f;

    for (int g = g0; g < g0 + ng; ++g) {
        const size_t blk = (size_t)t * G + g;
        const int z = (int)((Z[blk * kZBlockWords + (col >> 3)] >> (4 * (col & 7))) & 15u);
        const float s = __half2float(S[blk * kSBlockHalves + col]);
        const uint32_t* wb = Wq + blk * kBlockWords;
        for (int kw = 0; kw < kGroup / 8; ++kw) {
            const uint32_t w = wb[block_word_index(col, kw)];
            const int k0 = g * kGroup + kw * 8;
#pragma unroll
            for (int p = 0; p < 8; ++p) {
                const int off = 2 * (p & 3) + (p >> 2);
                const int q = (int)((w >> (4 * p)) & 15u);
                const float w16 = __half2float(__float2half_rn((float)(q - z) * s));
#pragma unroll
                for (int mm = 0; mm < kSimpleMB; ++mm) {
                    if (m0 + mm < M)
                        acc[mm] = fmaf(__half2float(A[(size_t)(m0 + mm) * K + k0 + off]), w16, acc[mm]);
                }
            }
        }
    }
    const int n = t * kTileN + col;
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

// Diagnostic: one warp waits on a barrier that nobody ever arrives on, with a limit of `limit_ns`.  The wait
// runs out, records kStatusMbarTimeout in the status word and the kernel returns normally: the same exit
// every GEMM kernel takes when one of its waits gives up, exercised without any fault.
__global__ void wait_timeout_probe_kernel(unsigned long long limit_ns, int* gave_up) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        fence_mbar_init();
    }
    __syncthreads();
    const bool ok = mbar_wait(&bar, 0u, limit_ns);
    if (threadIdx.x == 0 && gave_up != nullptr) *gave_up = ok ? 0 : 1;
}

}  // namespace w4a16
