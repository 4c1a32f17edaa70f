// pack (offline reorder), standalone dequant, the plain FP32-FMA GEMM and the Split-K
// reduce kernel.
#pragma once

#include "common.cuh"

namespace w4a16 {

// ------------------------------------------------------------------ pack
// Decode a packed word's position: idx -> block, column inside the tile, first k inside the block.
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

// Scales: packed position idx = ((blk * sg + j) * 64 + sz_perm(col)); one thread per raw scale.
__global__ void pack_s_kernel(const uint16_t* __restrict__ raw, uint16_t* __restrict__ out, int N, int G, int sg,
                              size_t total) {
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;   // over (t, g, j, col)
    if (idx >= total) return;
    const int col = (int)(idx & 63);
    const size_t row = idx >> 6;                 // (t * G + g) * sg + j
    const int j = (int)(row % sg);
    const size_t blk = row / sg;
    const int t = (int)(blk / G), g = (int)(blk % G);
    out[row * kSBlockHalves + sz_perm(col)] = raw[(size_t)(g * sg + j) * N + (size_t)t * kTileN + col];
}

// Zero points: one thread per packed word (eight permuted positions of one row).
__global__ void pack_z_kernel(const uint8_t* __restrict__ raw, uint32_t* __restrict__ out, int N, int G, int sg,
                              size_t total_words) {
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total_words) return;
    const int wi = (int)(idx & 7);
    const size_t row = idx >> 3;
    const int j = (int)(row % sg);
    const size_t blk = row / sg;
    const int t = (int)(blk / G), g = (int)(blk % G);
    uint32_t w = 0;
    for (int col = 0; col < kTileN; ++col) {
        const int p = sz_perm(col);
        if ((p >> 3) == wi)
            w |= (uint32_t)(raw[(size_t)(g * sg + j) * N + (size_t)t * kTileN + col] & 15u) << (4 * (p & 7));
    }
    out[idx] = w;
}

// Scale (16-bit pattern) and zero point of column `col` for the k-word kw (0..15) of block blk.
__device__ __forceinline__ void load_sz(const uint16_t* __restrict__ S, const uint32_t* __restrict__ Z, size_t blk,
                                        int sg, int col, int kw, uint16_t& s, uint32_t& z) {
    const int j = (kw * 8) / (kGroup / sg);
    const size_t row = blk * sg + j;
    const int p = sz_perm(col);
    s = S[row * kSBlockHalves + p];
    z = Z == nullptr ? (uint32_t)kSymZero : ((Z[row * kZBlockWords + (p >> 3)] >> (4 * (p & 7))) & 15u);
}

// ------------------------------------------------------------------ quantize (the step before the path)
// Eq. 1, x_q = round(x / s) + z, per group of `group` consecutive k of one column: one thread per (group,
// column).  Asymmetric: s = (max - min) / 15 rounded to the 16-bit format, z = clamp(round(-min / s), 0, 15);
// symmetric: s = max|x| / 7, z = 8; a zero or non-finite s becomes 1; q = clamp(round(x / s) + z, 0, 15),
// ties to even.  Every operation is one IEEE binary32 operation in this order, because the results are
// integers decided by floating point.  Output in the raw layout that w4a16_pack consumes.
template <bool BF>
__device__ __forceinline__ float group_scale(float num, float den, uint16_t& bits) {
    bits = cast_out<BF>(__fdiv_rn(num, den));
    float s = widen<BF>(bits);
    if (!(s > 0.0f) || isinf(s)) {
        s = 1.0f;
        bits = cast_out<BF>(1.0f);
    }
    return s;
}

template <bool BF>
__global__ void quantize_kernel(const uint16_t* __restrict__ W16, uint32_t* __restrict__ Wq, uint16_t* __restrict__ S,
                                uint8_t* __restrict__ Z, int N, int G, int group, int symmetric) {
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;   // (g, n), n fastest
    if (idx >= (size_t)G * N) return;
    const int n = (int)(idx % (size_t)N), g = (int)(idx / (size_t)N);
    const uint16_t* col = W16 + (size_t)g * group * N + n;
    float lo = INFINITY, hi = -INFINITY, amax = 0.0f;
    for (int k = 0; k < group; ++k) {
        const float x = widen<BF>(col[(size_t)k * N]);
        lo = x < lo ? x : lo;
        hi = x > hi ? x : hi;
        amax = fabsf(x) > amax ? fabsf(x) : amax;
    }
    uint16_t sb;
    float s;
    int z;
    if (symmetric) {
        s = group_scale<BF>(amax, 7.0f, sb);
        z = kSymZero;
    } else {
        s = group_scale<BF>(__fsub_rn(hi, lo), 15.0f, sb);
        const float zf = rintf(__fdiv_rn(-lo, s));
        z = zf < 0.0f ? 0 : zf > 15.0f ? 15 : (int)zf;
    }
    S[idx] = sb;
    if (Z != nullptr) Z[idx] = (uint8_t)z;
    for (int kw = 0; kw < group / 8; ++kw) {
        uint32_t w = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float x = widen<BF>(col[(size_t)(kw * 8 + i) * N]);
            const float r = __fadd_rn(rintf(__fdiv_rn(x, s)), (float)z);
            const int q = r < 0.0f ? 0 : r > 15.0f ? 15 : (int)r;
            w |= (uint32_t)q << (4 * i);
        }
        Wq[((size_t)g * (group / 8) + kw) * N + n] = w;
    }
}

// ------------------------------------------------------------------ dequant
// Algorithm 1, Phase 1 as a standalone kernel: one thread per packed word, eight results
// w16 = rn((q - z) * s) in the 16-bit format: (q - z) is formed exactly and multiplied by s with one
// multiply (round-to-nearest-even, subnormals kept).  Z == nullptr: symmetric format, z = 8.
template <bool BF>
__global__ void dequant_kernel(const uint32_t* __restrict__ Wq, const uint16_t* __restrict__ S,
                               const uint32_t* __restrict__ Z, uint16_t* __restrict__ W16, int N, int G, int sg,
                               size_t total_words) {
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total_words) return;
    size_t blk;
    int col, kw;
    word_position(idx, blk, col, kw);
    const int t = (int)(blk / G), g = (int)(blk % G);
    uint16_t s;
    uint32_t z;
    load_sz(S, Z, blk, sg, col, kw, s, z);
    const Pack8 f = dequant_word<BF>(Wq[idx], zconst_lo<BF>(z), zconst_hi<BF>(z), (uint32_t)s * 0x00010001u);
    uint16_t* p = W16 + (size_t)(g * kGroup + kw * 8) * N + (size_t)t * kTileN + col;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        p[(size_t)(2 * j) * N] = (uint16_t)(f.h[j] & 0xffffu);
        p[(size_t)(2 * j + 1) * N] = (uint16_t)(f.h[j] >> 16);
    }
}

// ------------------------------------------------------------------ plain GEMM
// Correct-first kernel: one thread per output column of a 64-column tile, kSimpleMB batch
// rows per thread, FP32 FMA over this CTA's K-slice.  Grid: (N/64,
// ceil(M/kSimpleMB), split_k).  With split_k == 1 it writes C, else FP32 partials
// ws[split][M][N] (Algorithm 1, Phase 2) for splitk_reduce_kernel.
constexpr int kSimpleMB = 4;

__device__ __forceinline__ void slice_of(int G, int split_k, int sp, int& g0, int& ng) {
    int base = G / split_k, rem = G % split_k;
    g0 = sp * base + min(sp, rem);
    ng = base + (sp < rem ? 1 : 0);
}

template <bool BF>
__global__ void __launch_bounds__(64)
gemm_simple_kernel(const uint16_t* __restrict__ A, const uint32_t* __restrict__ Wq, const uint16_t* __restrict__ S,
                   const uint32_t* __restrict__ Z, uint16_t* __restrict__ C, float* __restrict__ ws, int M, int N,
                   int K, int G, int sg, int split_k, Epilogue epi) {
    const int t = blockIdx.x, m0 = blockIdx.y * kSimpleMB, sp = blockIdx.z;
    const int col = threadIdx.x;  // column inside the tile
    int g0, ng;
    slice_of(G, split_k, sp, g0, ng);

    float acc[kSimpleMB];
#pragma unroll
    for (int i = 0; i < kSimpleMB; ++i) acc[i] = 0.f;

    for (int g = g0; g < g0 + ng; ++g) {
        const size_t blk = (size_t)t * G + g;
        const uint32_t* wb = Wq + blk * kBlockWords;
        for (int kw = 0; kw < kGroup / 8; ++kw) {
            uint16_t sb;
            uint32_t z;
            load_sz(S, Z, blk, sg, col, kw, sb, z);
            const float s = widen<BF>(sb);
            const uint32_t w = wb[block_word_index(col, kw)];
            const int k0 = g * kGroup + kw * 8;
#pragma unroll
            for (int p = 0; p < 8; ++p) {
                const int off = 2 * (p & 3) + (p >> 2);
                const int q = (int)((w >> (4 * p)) & 15u);
                // (q - z) * s is exact in FP32; one rounding to the 16-bit format, as in Phase 1
                const float w16 = widen<BF>(cast_out<BF>((float)(q - (int)z) * s));
#pragma unroll
                for (int mm = 0; mm < kSimpleMB; ++mm) {
                    if (m0 + mm < M)
                        acc[mm] = fmaf(widen<BF>(A[(size_t)(m0 + mm) * K + k0 + off]), w16, acc[mm]);
                }
            }
        }
    }
    const int n = t * kTileN + col;
#pragma unroll
    for (int mm = 0; mm < kSimpleMB; ++mm) {
        if (m0 + mm < M) {
            if (split_k == 1)
                C[(size_t)(m0 + mm) * N + n] = finish<BF>(acc[mm], n, epi);
            else
                ws[((size_t)sp * M + m0 + mm) * N + n] = acc[mm];
        }
    }
}

// Algorithm 1, Phase 3: C = rn16(sum_{i<S} C_i), ascending i, FP32.
template <bool BF>
__global__ void splitk_reduce_kernel(const float* __restrict__ ws, uint16_t* __restrict__ C, size_t MN, int N,
                                     int split_k, Epilogue epi) {
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= MN) return;
    float acc = ws[i];
    for (int s = 1; s < split_k; ++s) acc += ws[(size_t)s * MN + i];
    C[i] = finish<BF>(acc, (int)(i % (size_t)N), epi);
}

// Algorithm 1, Phase 3 for the tcgen05 kernel when every column tile is cut into `split_k` slices of its own
// CTAs: that kernel only stores its FP32 partial tiles (slot 2 (T split_k + s) of [batch row in tile][128
// columns]) and this one, launched behind it, sums them in ascending s, applies the optional bias /
// activation and rounds once.  A thread takes four neighbouring columns of one batch row.  Inside the GEMM
// kernel the same sum was a chain of L2 round trips in the one CTA per tile that finished last (5 to 10 us
// of a 32 us launch at M = 256); here the whole GPU does it at once.
template <bool BF>
__global__ void __launch_bounds__(256)
tile_splitk_reduce_kernel(const float* __restrict__ ws, uint16_t* __restrict__ C, int M, int N, int mt_log2, int n_tiles,
                          int split_k, long long quads, Epilogue epi) {
    // the next kernel of the stream may start its prologue; the partial tiles are the previous kernel's output
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= quads) return;
    const int mt = 1 << mt_log2;
    const int nq = (int)(q & 31);                       // which four of the tile's 128 columns
    const long long r = q >> 5;
    const int m_local = (int)(r & (mt - 1));
    const int T = (int)(r >> mt_log2);                  // tile = batch tile * n_tiles + column tile
    const int mt_i = T / n_tiles, nt = T - mt_i * n_tiles;
    const int m = mt_i * mt + m_local, n = nt * 128 + nq * 4;
    if (m >= M || n >= N) return;
    const size_t slot = (size_t)2 * mt * 128;           // floats between the slots of neighbouring slices
    const float* src = ws + ((size_t)T * split_k) * slot + (size_t)m_local * 128 + nq * 4;
    float4 acc = __ldcg(reinterpret_cast<const float4*>(src));
    int s = 1;
    for (; s + 3 < split_k; s += 4) {                   // four slices' loads in flight, added in order
        const float4 x0 = __ldcg(reinterpret_cast<const float4*>(src + (size_t)s * slot));
        const float4 x1 = __ldcg(reinterpret_cast<const float4*>(src + (size_t)(s + 1) * slot));
        const float4 x2 = __ldcg(reinterpret_cast<const float4*>(src + (size_t)(s + 2) * slot));
        const float4 x3 = __ldcg(reinterpret_cast<const float4*>(src + (size_t)(s + 3) * slot));
        acc.x += x0.x; acc.y += x0.y; acc.z += x0.z; acc.w += x0.w;
        acc.x += x1.x; acc.y += x1.y; acc.z += x1.z; acc.w += x1.w;
        acc.x += x2.x; acc.y += x2.y; acc.z += x2.z; acc.w += x2.w;
        acc.x += x3.x; acc.y += x3.y; acc.z += x3.z; acc.w += x3.w;
    }
    for (; s < split_k; ++s) {
        const float4 x = __ldcg(reinterpret_cast<const float4*>(src + (size_t)s * slot));
        acc.x += x.x; acc.y += x.y; acc.z += x.z; acc.w += x.w;
    }
    const uint32_t lo = (uint32_t)finish<BF>(acc.x, n, epi) | ((uint32_t)finish<BF>(acc.y, n + 1, epi) << 16);
    const uint32_t hi = (uint32_t)finish<BF>(acc.z, n + 2, epi) | ((uint32_t)finish<BF>(acc.w, n + 3, epi) << 16);
    *reinterpret_cast<uint2*>(C + (size_t)m * N + n) = make_uint2(lo, hi);
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
