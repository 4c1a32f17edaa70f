// Tensor-core tile kernel of the W4A16 GEMM: tcgen05.mma with the accumulator in tensor memory.
//
// The product is computed transposed, C^T[n, m] = sum_k W16[k, n] A[m, k], so that the
// DEQUANTIZED WEIGHTS are the MMA's 128-row A operand and live only in tensor memory:
//
//   HBM --TMA bulk--> shared (packed nibbles, scales, zeros)          producer warp
//   shared -> registers: unpack, (q - z) exact, * s in FP16            8 dequant warps
//   registers --tcgen05.st--> TMEM (A operand, one column n per lane, k packed along columns)
//   HBM --TMA tensor (128B swizzle)--> shared (activation tile, MT rows m x 64 k): B operand
//   tcgen05.mma.kind::f16  D[128 n x MT m] (FP32, TMEM) += A(TMEM) . B(shared)   one thread
//   TMEM --tcgen05.ld--> registers -> FP16 C, or FP32 partial tile + ticket (Split-K)
//
// so dequantized weights never touch shared or global memory (Algorithm 1's Phase 1 output
// stays on chip), and the activation tile is re-used by all 128 columns of the CTA tile.
//
// A work item is (column tile of 128 n, batch tile of MT m, K slice of whole groups); items are
// dealt round-robin to a persistent grid.  One pipeline stage is 64 k: 4 KiB of nibbles, the
// group's scales and zeros, and an MT x 64 FP16 activation box.  The two sets of four dequant
// warps take alternate stages; inside a set warp w owns TMEM lanes 32 (w % 4) .. + 31, one
// column n per thread.  All waits are bounded mbarrier waits; a wait that runs out records a
// status code and the CTA drains and exits (TMEM is always released).
#pragma once

#include <cuda.h>

#include "common.cuh"

namespace w4a16 {

constexpr int kTileCols = 128;                      // n per CTA tile = UMMA M
constexpr int kTileStageK = 64;                     // k per pipeline stage
constexpr int kTileDequantWarps = 8;
constexpr int kTileThreads = (2 + kTileDequantWarps) * 32;   // producer, MMA, 8 dequant/epilogue warps
constexpr int kTileASlots = 8;                      // TMEM ring of A-operand slots (32 columns each)
constexpr int kTileAColBase = 256;                  // D occupies columns [0, MT), the ring [256, 512)
constexpr int kTileStageW = 0;                      // 2 x 2 KiB of nibbles (two 64-column packed tiles)
constexpr int kTileStageS = 4096;                   // 2 x 64 FP16
constexpr int kTileStageZ = 4352;                   // 2 x 8 uint32
constexpr int kTileStageAct = 5120;                 // MT x 128 B, 1024-byte aligned (128B swizzle atom)
constexpr int kTileMaxStages = 8;
constexpr int kTileBarBytes = 1024;

__host__ __device__ constexpr int tile_stage_bytes(int mt) { return kTileStageAct + mt * 128; }

struct TileParams {
    const uint32_t* Wq;
    const __half* S;
    const uint32_t* Z;
    __half* C;
    float* ws;       // Split-K partial tiles [item][MT][128] FP32
    int* tickets;    // zeroed counters, eight (one per epilogue warp) per (column tile, batch tile)
    int M, N, K, G;
    int n_tiles;     // ceil(N / 128)
    int m_tiles;     // ceil(M / MT)
    int split_k;     // >= 1
    int stages;
};

// ------------------------------------------------------------------ tcgen05 / TMA wrappers
__device__ __forceinline__ void tma_load_2d(void* smem_dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(smem_dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar))
        : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}
// D(tmem) (+)= A(tmem) . B(shared descriptor); `accumulate` == 0 overwrites D.
__device__ __forceinline__ void tc_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// 32 consecutive 32-bit TMEM columns of this thread's lane <- registers.
__device__ __forceinline__ void tc_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
        "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
        "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
        "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
        "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major operand tile stored as 128-byte rows with the
// 128-byte swizzle (what the activation TMA writes): 8-row groups are 1024 B apart, the
// leading-dimension offset is unused for a tile one swizzle atom wide, descriptor version 1,
// layout code 2 = 128-byte swizzle.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;                    // leading byte offset (ignored for swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;          // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                    // descriptor version
    d |= (uint64_t)2 << 61;                    // SWIZZLE_128B
    return d;
}

// kind::f16 instruction descriptor: FP32 accumulator, FP16 A and B, both K-major, M = 128, N = mt.
__host__ __device__ constexpr uint32_t tile_idesc(int mt) {
    return (1u << 4) | ((uint32_t)(mt >> 3) << 17) | ((uint32_t)(kTileCols >> 4) << 24);
}

// K slice `sp` of `split_k` over G groups: first group and count (first G % split_k slices get one more).
__device__ __forceinline__ void tile_slice(int G, int split_k, int sp, int& g0, int& ng) {
    const int base = G / split_k, rem = G % split_k;
    g0 = sp * base + min(sp, rem);
    ng = base + (sp < rem ? 1 : 0);
}

template <int MT>
__global__ void __launch_bounds__(kTileThreads, 1)
gemm_tile_kernel(const __grid_constant__ CUtensorMap tmap_a, const TileParams p) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    // 1024-byte alignment of the stage buffers (the swizzle atom) regardless of where the
    // dynamic segment starts
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    constexpr int kStageBytes = tile_stage_bytes(MT);
    constexpr uint32_t kIdesc = tile_idesc(MT);
    constexpr int kColsPerWarp = MT / 2;      // epilogue: two warps share a lane quarter

    uint64_t* full = reinterpret_cast<uint64_t*>(smem);          // [stages]  TMA landed
    uint64_t* empty = full + kTileMaxStages;                     // [stages]  MMAs that read the stage retired
    uint64_t* a_full = empty + kTileMaxStages;                   // [slots]   dequantized operand stored
    uint64_t* a_empty = a_full + kTileASlots;                    // [slots]   MMAs that read the slot retired
    uint64_t* d_full = a_empty + kTileASlots;                    // accumulator complete
    uint64_t* d_empty = d_full + 1;                              // accumulator drained by the epilogue
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(d_empty + 1);
    int* flags = reinterpret_cast<int*>(tmem_slot + 1);          // [0] a bounded wait ran out, [1] stages issued
    unsigned char* stage0 = smem + kTileBarBytes;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int stages = p.stages;

    if (threadIdx.x == 0) {
        for (int i = 0; i < stages; ++i) {
            mbar_init(&full[i], 1);
            mbar_init(&empty[i], 1);
        }
        for (int i = 0; i < kTileASlots; ++i) {
            mbar_init(&a_full[i], 4);
            mbar_init(&a_empty[i], 1);
        }
        mbar_init(d_full, 1);
        mbar_init(d_empty, kTileDequantWarps);
        flags[0] = 0;
        flags[1] = 0;
        fence_mbar_init();
    }
    if (warp == 1) {
        // whole tensor memory of the SM: 512 columns (one CTA per SM by shared-memory size)
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(tmem_slot))
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    volatile int* abort_flag = flags;

    const int total_items = p.n_tiles * p.m_tiles * p.split_k;

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_a) : "memory");
            uint32_t n_stage = 0;
            bool ok = true;
            for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x) {
                const int mt_i = item % p.m_tiles;
                const int rest = item / p.m_tiles;
                const int sp = rest % p.split_k;
                const int nt = rest / p.split_k;
                int g0, ng;
                tile_slice(p.G, p.split_k, sp, g0, ng);
                const int t0 = 2 * nt;                          // packed 64-column tiles t0, t0 + 1
                const bool has_t1 = (t0 + 1) * kTileN < p.N;
                const uint32_t tx = (has_t1 ? 2u : 1u) * (2048u + 128u + 32u) + (uint32_t)MT * 128u;
                for (int st = 0; st < 2 * ng && ok; ++st, ++n_stage) {
                    const int slot = n_stage % stages;
                    const uint32_t ph = (n_stage / stages) & 1u;
                    if (!mbar_wait(&empty[slot], ph ^ 1u)) { ok = false; break; }
                    const int g = g0 + (st >> 1), c = st & 1;
                    unsigned char* sb = stage0 + (size_t)slot * kStageBytes;
                    mbar_expect_tx(&full[slot], tx);
                    for (int h = 0; h < (has_t1 ? 2 : 1); ++h) {
                        const size_t blk = (size_t)(t0 + h) * p.G + g;
                        bulk_g2s(sb + kTileStageW + h * 2048, p.Wq + blk * kBlockWords + c * 512, 2048, &full[slot]);
                        bulk_g2s(sb + kTileStageS + h * 128, p.S + blk * kSBlockHalves, 128, &full[slot]);
                        bulk_g2s(sb + kTileStageZ + h * 32, p.Z + blk * kZBlockWords, 32, &full[slot]);
                    }
                    tma_load_2d(sb + kTileStageAct, &tmap_a, g * kGroup + c * kTileStageK, mt_i * MT, &full[slot]);
                }
            }
            flags[1] = (int)n_stage;
            if (!ok) *abort_flag = 1;
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            uint32_t n_stage = 0, n_item = 0;
            bool ok = true;
            for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x, ++n_item) {
                const int sp = (item / p.m_tiles) % p.split_k;
                int g0, ng;
                tile_slice(p.G, p.split_k, sp, g0, ng);
                // the epilogue of the previous item must have drained the accumulator
                if (!mbar_wait(d_empty, (n_item & 1u) ^ 1u)) { ok = false; break; }
                tc_fence_after();
                for (int st = 0; st < 2 * ng; ++st, ++n_stage) {
                    const int slot = n_stage % stages;
                    const uint32_t ph = (n_stage / stages) & 1u;
                    const int aslot = n_stage % kTileASlots;
                    const uint32_t aph = (n_stage / kTileASlots) & 1u;
                    if (!mbar_wait(&full[slot], ph) || !mbar_wait(&a_full[aslot], aph)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t act = smem_u32(stage0 + (size_t)slot * kStageBytes + kTileStageAct);
                    const uint64_t bdesc = smem_desc_sw128(act);
                    const uint32_t a_t = tmem_base + kTileAColBase + aslot * 32;
#pragma unroll
                    for (int kk = 0; kk < kTileStageK / 16; ++kk) {
                        // 16 k per instruction: 8 TMEM columns of A, 32 bytes along the swizzled rows of B
                        tc_mma_ts(tmem_base, a_t + kk * 8, bdesc + (uint64_t)(kk * 2), kIdesc, (st | kk) != 0 ? 1u : 0u);
                    }
                    tc_commit(&empty[slot]);
                    tc_commit(&a_empty[aslot]);
                }
                if (ok) tc_commit(d_full);
            }
            if (!ok) *abort_flag = 1;
        }
    } else {
        // ------------------------------------------------------------ dequant + epilogue warps
        const int dw = warp - 2;               // 0..7
        const int set = dw >> 2;               // stages with (index & 1) == set
        const int quarter = warp & 3;          // TMEM lanes this warp may touch
        const int row = quarter * 32 + lane;   // column n inside the CTA tile = TMEM lane
        const int half = row >> 6, col = row & 63;
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        // this thread's two 16-byte chunks of a 64-k line pair
        const int woff0 = half * 2048 + (col >> 3) * 256 + (col & 7) * 16;
        const int woff1 = half * 2048 + (col >> 3) * 256 + 128 + (((col & 7) + 4) & 7) * 16;
        uint32_t n_stage = 0, n_item = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x, ++n_item) {
            const int mt_i = item % p.m_tiles;
            const int rest = item / p.m_tiles;
            const int sp = rest % p.split_k;
            const int nt = rest / p.split_k;
            int g0, ng;
            tile_slice(p.G, p.split_k, sp, g0, ng);
            for (int st = 0; st < 2 * ng; ++st, ++n_stage) {
                if ((int)(n_stage & 1u) != set) continue;
                const int slot = n_stage % stages;
                const uint32_t ph = (n_stage / stages) & 1u;
                const int aslot = n_stage % kTileASlots;
                const uint32_t aph = (n_stage / kTileASlots) & 1u;
                if (!mbar_wait(&full[slot], ph) || !mbar_wait(&a_empty[aslot], aph ^ 1u)) { ok = false; break; }
                tc_fence_after();
                const unsigned char* sb = stage0 + (size_t)slot * kStageBytes;
                const uint4 w0 = *reinterpret_cast<const uint4*>(sb + kTileStageW + woff0);
                const uint4 w1 = *reinterpret_cast<const uint4*>(sb + kTileStageW + woff1);
                const __half s = *reinterpret_cast<const __half*>(sb + kTileStageS + row * 2);
                const uint32_t zw = *reinterpret_cast<const uint32_t*>(sb + kTileStageZ + (row >> 3) * 4);
                const uint32_t z = (zw >> (4 * (row & 7))) & 15u;
                const __half2 s2 = __half2half2(s);
                const __half2 zlo = u32_as_h2(zmagic_lo(z)), zhi = u32_as_h2(zmagic_hi(z));
                const uint32_t ww[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
                uint32_t regs[32];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const Half8 f = dequant_word(ww[i], zlo, zhi, s2);
#pragma unroll
                    for (int j = 0; j < 4; ++j) regs[4 * i + j] = h2_as_u32(f.h[j]);
                }
                tc_st32(tmem_base + lane_addr + kTileAColBase + aslot * 32, regs);
                tc_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&a_full[aslot]);
            }
            if (!ok) break;

            // ---------------------------------------------------- epilogue of this item
            if (!mbar_wait(d_full, n_item & 1u)) { ok = false; break; }
            tc_fence_after();
            const int n = nt * kTileCols + row;
            const int m_base = mt_i * MT;
            const int col0 = set * kColsPerWarp;    // this warp's share of the accumulator columns
            if (p.split_k == 1) {
#pragma unroll 1
                for (int cc = 0; cc < kColsPerWarp; cc += 16) {
                    uint32_t v[16];
                    tc_ld16(tmem_base + lane_addr + col0 + cc, v);
                    tc_wait_ld();
                    if (n < p.N) {
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const int m = m_base + col0 + cc + j;
                            if (m < p.M) p.C[(size_t)m * p.N + n] = __float2half_rn(__uint_as_float(v[j]));
                        }
                    }
                }
            } else {
                float* slot_ws = p.ws + (size_t)item * (MT * kTileCols);
#pragma unroll 1
                for (int cc = 0; cc < kColsPerWarp; cc += 16) {
                    uint32_t v[16];
                    tc_ld16(tmem_base + lane_addr + col0 + cc, v);
                    tc_wait_ld();
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        slot_ws[(size_t)(col0 + cc + j) * kTileCols + row] = __uint_as_float(v[j]);
                }
            }
            // accumulator drained: the next item's first MMA may overwrite it
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(d_empty);

            if (p.split_k > 1) {
                // Split-K reduce (Algorithm 1, Phase 3), per warp region (32 columns n x MT/2 rows m): the
                // warp that draws the region's last ticket adds the S partial regions in ascending slice
                // order and casts to FP16.  No warp waits for another CTA.
                __threadfence();
                __syncwarp();
                int* ticket = p.tickets + ((size_t)(nt * p.m_tiles + mt_i) * kTileDequantWarps + dw);
                int last = 0;
                if (lane == 0) {
                    const int old = atomicAdd(ticket, 1);
                    last = (old == p.split_k - 1);
                    if (last) *ticket = 0;   // every contributor has arrived: zero for the next call
                }
                last = __shfl_sync(0xffffffffu, last, 0);
                if (last) {
                    __threadfence();
                    // items of this tile: ((nt * split_k + s) * m_tiles + mt_i), s = 0 .. split_k - 1
                    const float* base = p.ws + ((size_t)nt * p.split_k * p.m_tiles + mt_i) * (MT * kTileCols) + row;
                    const size_t s_stride = (size_t)p.m_tiles * (MT * kTileCols);
#pragma unroll 4
                    for (int mm = col0; mm < col0 + kColsPerWarp; ++mm) {
                        float acc = 0.f;
                        for (int s = 0; s < p.split_k; ++s) acc += __ldcg(base + s * s_stride + (size_t)mm * kTileCols);
                        const int m = m_base + mm;
                        if (m < p.M && n < p.N) p.C[(size_t)m * p.N + n] = __float2half_rn(acc);
                    }
                }
            }
        }
        if (!ok) *abort_flag = 1;
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (*abort_flag != 0 && threadIdx.x == 0) {
        // some wait ran out: before the CTA's shared memory goes away, give the copies still in
        // flight a (bounded) chance to land -- the last use of every stage slot
        const uint32_t issued = (uint32_t)flags[1];
        for (uint32_t back = 0; back < (uint32_t)stages && back < issued; ++back) {
            const uint32_t ns = issued - 1 - back;
            mbar_wait(&full[ns % stages], (ns / stages) & 1u);
        }
    }
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
    }
}

}  // namespace w4a16
