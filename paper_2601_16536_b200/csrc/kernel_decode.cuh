// Small-M ("decode") W4A16 GEMM: bandwidth-bound skinny GEMM.
//
// One CTA owns a 64-column tile of C and one Split-K slice of whole groups.  A producer
// warp streams the slice's packed blocks (16 KiB = 4 groups per stage, one TMA bulk copy)
// and the matching activation rows into a multi-stage shared-memory ring guarded by
// mbarriers.  Four consumer warps each take one group per stage: a 128-bit shared load
// gives a lane the A-fragment nibbles of a 16-row sub-tile, a logic op and two FP16 ops
// per register turn them into w16 = fp16_rn((q - z) s), and an m16n8k16 tensor-core MMA
// with the WEIGHTS as the 16-row operand (MMA rows = n, MMA columns = batch rows)
// accumulates in FP32.  The four warps' partial sums (disjoint k) are added in warp order
// through shared memory; the result goes to C (split_k == 1) or to the FP32 Split-K
// workspace.
#pragma once

#include "common.cuh"
#include "kernels_basic.cuh"

namespace w4a16 {

constexpr int kDecWarps = 4;                       // consumer warps = groups per stage
constexpr int kDecThreads = (kDecWarps + 1) * 32;  // + producer warp
constexpr int kDecStageW = kDecWarps * kBlockBytes;             // 16 KiB of packed weights
constexpr int kDecARowBytes = kDecWarps * kGroup * 2 + 16;      // 1024 B of k + 16 B pad
constexpr int kDecRedStride = 68;                  // floats per batch row in the reduce buffer

struct DecodeParams {
    const __half* A;
    const uint32_t* Wq;
    const __half* S;
    const uint32_t* Z;
    __half* C;
    float* ws;       // FP32 partials [split_k][M][N] when split_k > 1
    int M, N, K, G;
    int split_k;
    int stages;
    int sz_bytes;    // shared bytes reserved for the slice's scales + zeros (multiple of 128)
};

__host__ __device__ inline int decode_stage_bytes(int rows) { return kDecStageW + rows * kDecARowBytes; }

__device__ __forceinline__ void mma_m16n8k16(float (&d)[4], const Frag4& a, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(h2_as_u32(a.lo_a)), "r"(h2_as_u32(a.hi_a)), "r"(h2_as_u32(a.lo_b)), "r"(h2_as_u32(a.hi_b)),
          "r"(b0), "r"(b1));
}

// MB = number of 8-row batch blocks one CTA handles (rows m0 .. m0 + 8 MB - 1).
template <int MB>
__global__ void __launch_bounds__(kDecThreads) gemm_decode_kernel(const DecodeParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    const int t = blockIdx.x, sp = blockIdx.y;
    const int m0 = blockIdx.z * (8 * MB);
    const int rows = min(8 * MB, p.M - m0);  // batch rows this CTA really has
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int stages = p.stages;

    int g0, ng;
    slice_of(p.G, p.split_k, sp, g0, ng);
    const int n_iter = (ng + kDecWarps - 1) / kDecWarps;

    // shared layout: [barriers 128 B][S slice | Z slice][stage 0][stage 1]...
    uint64_t* full = reinterpret_cast<uint64_t*>(smem);
    uint64_t* empty = full + 6;
    uint64_t* szbar = full + 12;
    unsigned char* sz = smem + 128;
    const __half* s_s = reinterpret_cast<const __half*>(sz);
    const uint32_t* z_s = reinterpret_cast<const uint32_t*>(sz + ng * (kSBlockHalves * 2));
    unsigned char* stage0 = sz + p.sz_bytes;
    const int stage_bytes = decode_stage_bytes(8 * MB);

    if (threadIdx.x == 0) {
        for (int i = 0; i < stages; ++i) {
            mbar_init(&full[i], 1);
            mbar_init(&empty[i], kDecWarps);
        }
        mbar_init(szbar, 1);
        fence_mbar_init();
    }
    __syncthreads();

    const size_t blk0 = (size_t)t * p.G + g0;  // first packed block of the slice

    if (warp == kDecWarps) {
        // ------------------------------------------------ producer warp
        if (lane == 0) {
            mbar_expect_tx(szbar, (uint32_t)(ng * (kSBlockHalves * 2 + kZBlockWords * 4)));
            bulk_g2s(sz, p.S + blk0 * kSBlockHalves, (uint32_t)(ng * kSBlockHalves * 2), szbar);
            bulk_g2s(sz + ng * (kSBlockHalves * 2), p.Z + blk0 * kZBlockWords, (uint32_t)(ng * kZBlockWords * 4),
                     szbar);
        }
        for (int it = 0; it < n_iter; ++it) {
            const int s = it % stages;
            const int gc = min(kDecWarps, ng - it * kDecWarps);
            bool ok = true;
            if (it >= stages) ok = mbar_wait(&empty[s], (uint32_t)((it / stages - 1) & 1));
            if (!ok) break;  // status recorded; consumers will time out too and the CTA ends
            unsigned char* st = stage0 + (size_t)s * stage_bytes;
            if (lane == 0) {
                mbar_expect_tx(&full[s], (uint32_t)(gc * kBlockBytes + rows * gc * (kGroup * 2)));
                bulk_g2s(st, p.Wq + (blk0 + (size_t)it * kDecWarps) * kBlockWords, (uint32_t)(gc * kBlockBytes),
                         &full[s]);
            }
            __syncwarp();
            for (int m = lane; m < rows; m += 32) {
                bulk_g2s(st + kDecStageW + m * kDecARowBytes,
                         p.A + (size_t)(m0 + m) * p.K + (size_t)(g0 + it * kDecWarps) * kGroup,
                         (uint32_t)(gc * kGroup * 2), &full[s]);
            }
        }
        return;
    }

    // ---------------------------------------------------- consumer warps
    const int gq = lane >> 2, tig = lane & 3;
    float acc[4][MB][4];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int mb = 0; mb < MB; ++mb)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[r][mb][i] = 0.f;

    bool alive = mbar_wait(szbar, 0);

    for (int it = 0; it < n_iter && alive; ++it) {
        const int s = it % stages;
        alive = mbar_wait(&full[s], (uint32_t)((it / stages) & 1));
        if (!alive) break;
        const int gc = min(kDecWarps, ng - it * kDecWarps);
        if (warp < gc) {
            const int lg = it * kDecWarps + warp;  // group index inside the slice
            const unsigned char* st = stage0 + (size_t)s * stage_bytes;
            const uint4* wsm = reinterpret_cast<const uint4*>(st + warp * kBlockBytes);
            const unsigned char* asm_ = st + kDecStageW + warp * (kGroup * 2);

            // scales / zero points of this lane's 8 rows (16r + gq + 8h)
            uint4 sraw = *reinterpret_cast<const uint4*>(s_s + lg * kSBlockHalves + gq * 8);
            const uint32_t zw = z_s[lg * kZBlockWords + gq];
            const uint32_t sw[4] = {sraw.x, sraw.y, sraw.z, sraw.w};

            __half2 s_lo[4], s_hi[4], zlo[4], zhi[4];
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                s_lo[r] = __half2half2(__low2half(u32_as_h2(sw[r])));   // row 16r + gq
                s_hi[r] = __half2half2(__high2half(u32_as_h2(sw[r])));  // row 16r + gq + 8
                zlo[r] = u32_as_h2(zmagic_lo((zw >> (8 * r)) & 15u));
                zhi[r] = u32_as_h2(zmagic_hi((zw >> (8 * r + 4)) & 15u));
            }

#pragma unroll
            for (int c = 0; c < 2; ++c) {
                // B fragments: batch row 8 mb + gq, 16 consecutive k per lane
                uint32_t bw[MB][8];
#pragma unroll
                for (int mb = 0; mb < MB; ++mb) {
                    if (mb * 8 + gq < rows) {
                        const uint4* ap =
                            reinterpret_cast<const uint4*>(asm_ + (mb * 8 + gq) * kDecARowBytes + c * 128 + tig * 32);
                        uint4 x = ap[0], y = ap[1];
                        bw[mb][0] = x.x; bw[mb][1] = x.y; bw[mb][2] = x.z; bw[mb][3] = x.w;
                        bw[mb][4] = y.x; bw[mb][5] = y.y; bw[mb][6] = y.z; bw[mb][7] = y.w;
                    } else {
#pragma unroll
                        for (int i = 0; i < 8; ++i) bw[mb][i] = 0u;
                    }
                }
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    const uint4 wv = wsm[(c * 4 + r) * 32 + lane];
                    const uint32_t ww[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const Frag4 f = dequant_word(ww[j], zlo[r], zhi[r], s_lo[r], s_hi[r]);
#pragma unroll
                        for (int mb = 0; mb < MB; ++mb) mma_m16n8k16(acc[r][mb], f, bw[mb][2 * j], bw[mb][2 * j + 1]);
                    }
                }
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty[s]);
    }

    // ---------------------------------------------------- cross-warp sum (fixed order)
    // All copies this CTA issued have been consumed, so stage memory is free to reuse.
    float* red = reinterpret_cast<float*>(stage0);
    constexpr int kRows = 8 * MB;
    asm volatile("bar.sync 1, %0;" ::"n"(kDecWarps * 32) : "memory");
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int mb = 0; mb < MB; ++mb)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                int n = r * 16 + gq + (i >= 2 ? 8 : 0);
                int m = mb * 8 + 2 * tig + (i & 1);
                red[(warp * kRows + m) * kDecRedStride + n] = acc[r][mb][i];
            }
    asm volatile("bar.sync 1, %0;" ::"n"(kDecWarps * 32) : "memory");
    if (!alive) return;
    for (int idx = threadIdx.x; idx < rows * kTileN; idx += kDecWarps * 32) {
        int n = idx & (kTileN - 1), m = idx >> 6;
        float v = red[m * kDecRedStride + n];
#pragma unroll
        for (int w = 1; w < kDecWarps; ++w) v += red[(w * kRows + m) * kDecRedStride + n];
        size_t off = (size_t)(m0 + m) * p.N + (size_t)t * kTileN + n;
        if (p.split_k == 1)
            p.C[off] = __float2half_rn(v);
        else
            p.ws[(size_t)sp * p.M * p.N + off] = v;
    }
}

}  // namespace w4a16
