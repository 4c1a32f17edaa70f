// Small-M ("decode") W4A16 GEMM: a persistent, bandwidth-bound skinny GEMM.
//
// Work is counted in units: one unit = one packed block = 64 columns x one group (128 k),
// numbered u = tile * G + group, which is also the block's position in the packed buffers.
// The unit range [0, T*G) is cut into chunks; a CTA streams its chunk(s) front to back:
//   - balanced mode (split_k == 0): as many chunks as CTAs, equal to within one unit, so a
//     chunk may start and end in the middle of a column tile's K range;
//   - classic Split-K (split_k = S): every tile's K range is cut into S slices of whole
//     groups (Algorithm 1, Phase 2), T*S chunks dealt round-robin to the CTAs.
// A producer warp brings 4 units per stage (16 KiB of nibbles + their scales and zeros,
// three TMA bulk copies) plus the matching activation rows (one bulk copy per row, or one
// tensor copy for all of them: ABOX below) into a shared-memory ring guarded by mbarriers;
// stages never straddle a tile.  Eight consumer warps work on a
// stage, two per unit, each on two of the block's four 16-column sub-tiles: two 64-bit shared
// loads give a lane the nibbles of columns gq and gq + 8 at its 16 k, a logic op and two FP16
// ops per register turn them into w16 = fp16_rn((q - z) s), and an m16n8k16 tensor-core MMA
// with the WEIGHTS as the 16-row operand (MMA rows = n, MMA columns = batch rows) accumulates
// in FP32.
//
// When a CTA leaves a tile it adds its warps' sums in a fixed order through shared
// memory.  If it covered the tile's whole K range it writes FP16 C.  Otherwise it stores
// the FP32 partial tile in its workspace slot, fences and draws a ticket from the tile's
// counter; the CTA that draws the last ticket adds the partial tiles in ascending K order,
// casts to FP16 and writes C (Algorithm 1, Phase 3, inside the same launch).  No CTA
// waits for another one, and the order of the sum does not depend on which CTA comes
// last, so results are bit-identical from run to run.  Where the S slices of a tile each
// have a CTA and S <= 4, the launch is made of clusters of S CTAs and the partial tiles go
// through the first CTA's shared memory instead (template parameter CL below): same order
// of the sum, same bits, about half the latency.
#pragma once

#include "common.cuh"

namespace w4a16 {

constexpr int kDecUnitsPerStage = 4;
constexpr int kDecWarps = 8;                       // consumer warps (2 per unit of a stage)
constexpr int kDecConsumers = kDecWarps * 32;
constexpr int kDecThreads = kDecConsumers + 32;    // + producer warp
constexpr int kDecMaxStages = 6;
constexpr int kDecStageW = kDecUnitsPerStage * kBlockBytes;                 // 16384: nibbles
constexpr int kDecStageS = kDecStageW;                                      // scale rows start here
constexpr int kDecARowBytes = kDecUnitsPerStage * kGroup * 2 + 16;          // 1024 B of k + 16 B pad
constexpr int kDecRedStride = 68;                  // floats per batch row in the reduce buffer
// stage layout for SG scale rows per block: [4 x 4096 nibbles][4 x SG x 128 scales][4 x SG x 32 zeros][A rows]
__host__ __device__ constexpr int dec_stage_z(int sg) { return kDecStageS + kDecUnitsPerStage * sg * kSBlockHalves * 2; }
__host__ __device__ constexpr int dec_stage_a(int sg) { return dec_stage_z(sg) + kDecUnitsPerStage * sg * kZBlockWords * 4; }
__host__ __device__ constexpr int dec_unit_bytes(int sg, bool sym) {
    return kBlockBytes + sg * kSBlockHalves * 2 + (sym ? 0 : sg * kZBlockWords * 4);
}

struct DecodeParams {
    const uint16_t* A;
    const uint32_t* Wq;
    const uint16_t* S;
    const uint32_t* Z;  // nullptr: symmetric format, zero point 8
    uint16_t* C;
    float* ws;          // partial tiles: [m chunk][2 * nchunks slots][8 MB rows][64] FP32
    int* tickets;       // zeroed counters: [m chunk][T]
    int M, N, K, G, T;  // G = K / 128 blocks along K, T = N / 64 column tiles
    int split_k;        // 0: balanced chunks; S >= 1: classic Split-K
    int nchunks;        // balanced: gridDim.x; classic: T * split_k
    int stages;
    int stage_bytes;    // ring stride: decode_stage_bytes(rows of a batch chunk, sg)
    int prefetch;       // stages whose weights are requested before the wait for the previous kernel
    // chunk arithmetic, prepared by the host (decode_fill_chunk_math)
    FastDiv div_G, div_split, div_nchunks;
    int slice_base, slice_rem;   // classic: G / split_k, G % split_k
    int bal_q, bal_r;            // balanced: (T G) / nchunks, (T G) % nchunks
    Epilogue epi;
};

inline void decode_fill_chunk_math(DecodeParams& p) {
    p.div_G = fast_div_make((uint32_t)p.G);
    p.div_split = fast_div_make((uint32_t)(p.split_k > 0 ? p.split_k : 1));
    p.div_nchunks = fast_div_make((uint32_t)p.nchunks);
    p.slice_base = p.split_k > 0 ? p.G / p.split_k : 0;
    p.slice_rem = p.split_k > 0 ? p.G % p.split_k : 0;
    const long long units = (long long)p.T * p.G;
    p.bal_q = (int)(units / p.nchunks);
    p.bal_r = (int)(units % p.nchunks);
}

// Activation rows of a stage, two ways (template parameter ABOX of the kernel).  Few rows: one bulk copy per row into the tail of the weight stage
// (1 KiB + 16 B apart).  More rows: every bulk copy costs the producer warp about 50 clocks whatever its
// size, and 19 of them per 16 KiB stage leave the first ring-full a microsecond late; so the rows then come
// as ONE tensor copy (A seen as [K / 64][M][64], box = 8 chunks x 8 MB rows x 64 k, 128-byte swizzle, rows
// past M read as zero) into a second ring of 8 MB KiB slots, 1024-byte aligned, behind the weight ring.
constexpr int kDecABoxChunks = 2 * kDecUnitsPerStage;    // 64-k chunks per stage
__host__ __device__ constexpr int dec_a_box_bytes(int mb) { return kDecABoxChunks * 8 * mb * 128; }

// One ring stage holds the activation rows a CTA really has (min(M, 8 MB)), not 8 MB of them: a call with
// one batch row gets five stages where eight rows get four.  A multiple of 128 bytes, so that every
// stage starts on the same shared-memory bank.
__host__ __device__ inline int decode_stage_bytes(int rows, int sg, bool a_box = false) {
    return (dec_stage_a(sg) + (a_box ? 0 : rows * kDecARowBytes) + 127) / 128 * 128;
}
__host__ __device__ inline int decode_red_bytes(int mb) {
    return kDecUnitsPerStage * 8 * mb * kDecRedStride * 4;
}
// cluster exchange buffer (CL kernels): one partial tile of 8 mb rows x 64 columns per slice, at most
// kDecMaxCluster slices (clusters of 8 are the largest every device places, but measured worse than
// 6 everywhere: 6.5 against 6.0 us at K = 8192 / N = 2048, 18.8 against 9.2 with two batch blocks)
constexpr int kDecMaxCluster = 6;
// (the first CTA of a cluster keeps its own slice where it is: S - 1 slots)
__host__ __device__ inline int decode_xch_bytes(int mb, int slices) {
    return slices > 1 ? (slices - 1) * 8 * mb * kTileN * 4 : 0;
}
// Cluster kernels put the reduce buffer on top of the (by then idle) ring: a CTA of a cluster has one
// slice of one tile, so nothing is in flight when it leaves the tile.  The others leave tiles in
// mid-stream, with later stages already on their way, and keep a buffer of their own.
__host__ __device__ inline int decode_smem_bytes(int mb, int rows, int sg, int stages, int cluster_slices,
                                                 bool a_box = false) {
    // (a_box: the second ring and up to 1023 bytes in front of it for its alignment)
    const int ring = stages * decode_stage_bytes(rows, sg, a_box) + (a_box ? stages * dec_a_box_bytes(mb) + 1024 : 0);
    if (cluster_slices > 1) {
        const int r = decode_red_bytes(mb);
        return 128 + decode_xch_bytes(mb, cluster_slices) + (ring > r ? ring : r);
    }
    return 128 + decode_red_bytes(mb) + ring;
}

// D += A . B with A = (a0: row gq, a1: row gq + 8, a2 / a3: the same rows, second k pair).
template <bool BF>
__device__ __forceinline__ void mma_m16n8k16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                             uint32_t b0, uint32_t b1) {
    if constexpr (BF)
        asm volatile(
            "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
            "{%0,%1,%2,%3};"
            : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
            : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
    else
        asm volatile(
            "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
            "{%0,%1,%2,%3};"
            : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
            : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void consumer_bar() {
    asm volatile("bar.sync 1, %0;" ::"n"(kDecConsumers) : "memory");
}

// Shared-memory loads at a 32-bit shared address plus a compile-time offset: the per-stage base
// address is one register, everything else is an immediate.  (volatile + memory clobber keep them
// after the barrier wait that guards the stage.)
template <int OFF>
__device__ __forceinline__ uint2 lds64(uint32_t addr) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0, %1}, [%2 + %3];" : "=r"(v.x), "=r"(v.y) : "r"(addr), "n"(OFF) : "memory");
    return v;
}
template <int OFF>
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4 + %5];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "r"(addr), "n"(OFF)
                 : "memory");
    return v;
}
template <int OFF>
__device__ __forceinline__ uint32_t lds16(uint32_t addr) {
    uint32_t v;
    asm volatile("{\n\t.reg .b16 t;\n\tld.shared.u16 t, [%1 + %2];\n\tcvt.u32.u16 %0, t;\n\t}"
                 : "=r"(v) : "r"(addr), "n"(OFF) : "memory");
    return v;
}

// The producer's wait for a free ring slot.  It sleeps in the barrier unit between polls and is woken
// by every barrier event of the CTA, so the poll loop is kept to a few instructions: the wall-clock
// limit is checked only every 256th poll.
__device__ __forceinline__ bool mbar_wait_producer(uint64_t* bar, uint32_t parity) {
    const uint32_t addr = smem_u32(bar);
    unsigned long long t0 = 0;
    for (uint32_t it = 0;; ++it) {
        uint32_t ok;
        asm volatile(
            "{\n\t"
            ".reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t"
            "}"
            : "=r"(ok)
            : "r"(addr), "r"(parity), "r"(100000u)
            : "memory");
        if (ok) return true;
        if ((it & 255u) == 255u) {
            unsigned long long t1;
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
            if (t0 == 0) t0 = t1;
            else if (t1 - t0 > kWaitLimitNs) break;
        }
    }
    report_status(kStatusMbarTimeout);
    return false;
}

// First unit of chunk i (i == nchunks gives the end of the last chunk).
__device__ __forceinline__ int chunk_begin(const DecodeParams& p, int i) {
    // balanced: floor(i (T G) / nchunks) = i q + floor(i r / nchunks) with T G = q nchunks + r  (i r < nchunks^2)
    if (p.split_k == 0) return i * p.bal_q + fast_div(i * p.bal_r, p.div_nchunks);
    const int t = fast_div(i, p.div_split), s = i - t * p.split_k;
    return t * p.G + s * p.slice_base + min(s, p.slice_rem);
}
// The chunk that holds unit u.
__device__ __forceinline__ int chunk_of(const DecodeParams& p, int u) {
    if (p.split_k == 0) return (int)((((long long)u + 1) * p.nchunks - 1) / ((long long)p.T * p.G));
    const int t = u / p.G, g = u - t * p.G;
    const int base = p.G / p.split_k, rem = p.G % p.split_k;
    // slices 0..rem-1 hold base+1 groups, the rest base groups
    const int s = (g < rem * (base + 1)) ? g / (base + 1) : rem + (g - rem * (base + 1)) / max(base, 1);
    return t * p.split_k + s;
}

// The stages of a CTA in order: up to four consecutive units of one tile each.
struct DecStageIter {
    const DecodeParams& p;
    int ci, u, u1, t, tile_end;
    __device__ __forceinline__ DecStageIter(const DecodeParams& p_) : p(p_), ci((int)blockIdx.x), u(0), u1(0), t(0), tile_end(0) {
        load();
    }
    __device__ __forceinline__ void load() {
        while (ci < p.nchunks) {
            u = chunk_begin(p, ci);
            u1 = chunk_begin(p, ci + 1);
            if (u < u1) break;
            ci += (int)gridDim.x;
        }
        t = fast_div(u, p.div_G);
        tile_end = (t + 1) * p.G;
    }
    __device__ __forceinline__ bool valid() const { return ci < p.nchunks; }
    __device__ __forceinline__ int units() const { return min(kDecUnitsPerStage, min(u1, tile_end) - u); }
    __device__ __forceinline__ int group() const { return u - t * p.G; }
    __device__ __forceinline__ void next() {
        u += units();
        if (u == tile_end) { ++t; tile_end += p.G; }
        if (u >= u1) { ci += (int)gridDim.x; load(); }
    }
};

// MB = number of 8-row batch blocks one CTA handles (rows m0 .. m0 + 8 MB - 1); two CTAs per SM.
// CL: the launch is made of thread-block clusters of split_k CTAs, one cluster per column tile and
// one K slice per CTA (classic Split-K, every chunk on a CTA of its own).  The slices' partial tiles
// then meet in the shared memory of the cluster's first CTA (distributed shared memory + one
// hardware cluster barrier) instead of going through the workspace, a fence, a ticket and a reload:
// Phase 3 of Algorithm 1 in about a tenth of the time, still summed in ascending K order.
// SG = scale / zero-point rows per 128-k block (quantization group 128 / SG); BF = BF16 arithmetic;
// SYM = symmetric format (zero point 8, no Z buffer); ABOX = activation rows by tensor copy.
template <int MB, bool CL, int SG, bool BF, bool SYM, bool ABOX>
__global__ void __launch_bounds__(kDecThreads, 2) gemm_decode_kernel(const __grid_constant__ CUtensorMap tmap_a,
                                                                     const DecodeParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    constexpr int kRows = 8 * MB;
    constexpr int kStageZ = dec_stage_z(SG), kStageA = dec_stage_a(SG);
    const int stage_bytes = p.stage_bytes;
    constexpr bool sym = SYM;
    const int mz = blockIdx.y;
    const int m0 = mz * kRows;
    const int rows = min(kRows, p.M - m0);  // batch rows this CTA really has
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int stages = p.stages;

    // shared layout: [barriers + flag, 128 B][reduce buffer | exchange buffer (CL)][stage 0][stage 1]...
    // (CL: the reduce buffer lies on top of the ring, see decode_smem_bytes)
    uint64_t* full = reinterpret_cast<uint64_t*>(smem);
    uint64_t* empty = full + kDecMaxStages;
    uint64_t* xbar = full + 2 * kDecMaxStages;   // CL only: the other slices' partial tiles have landed (CTA 0's is used)
    int* last_flag = reinterpret_cast<int*>(smem + 120);
    float* xch = reinterpret_cast<float*>(smem + 128);   // CL only: [slice 1 .. S - 1][8 MB rows][64]
    unsigned char* stage0 = smem + 128 + (CL ? decode_xch_bytes(MB, p.split_k) : decode_red_bytes(MB));
    float* red = reinterpret_cast<float*>(CL ? stage0 : smem + 128);
    constexpr bool a_box = ABOX;
    constexpr uint32_t kABoxBytes = (uint32_t)dec_a_box_bytes(MB);
    // where the activation rows of slot 0 start, and the step to the next slot
    const uint32_t a_slot0 = a_box ? ((smem_u32(stage0) + (uint32_t)(stages * stage_bytes) + 1023u) & ~1023u)
                                   : smem_u32(stage0) + (uint32_t)kStageA;
    const uint32_t a_step = a_box ? kABoxBytes : (uint32_t)stage_bytes;

    if (threadIdx.x == 0) {
        for (int i = 0; i < stages; ++i) {
            mbar_init(&full[i], 1);
            mbar_init(&empty[i], kDecWarps);
        }
        if (CL) mbar_init(xbar, (uint32_t)((p.split_k - 1) * kDecWarps));   // one arrival per consumer warp of the other CTAs
        fence_mbar_init();
    }
    // (Batch rows this CTA does not have are never loaded: an MMA column only feeds its own output
    // column, and those columns are not stored.)
    __syncthreads();
    // CL: every CTA of the cluster must be running and have initialised its barriers before anyone writes to
    // another CTA's shared memory.  All threads of all CTAs of the cluster arrive here unconditionally (the
    // hardware launches a cluster's CTAs together), so the matching wait cannot hang; it stands where the
    // guarantee is needed, in front of the exchange (the barrier takes half a microsecond to complete, and
    // the producer warp has requests to make meanwhile).  Every other wait in this kernel is a bounded
    // mbarrier wait.
    // (relaxed: the barrier initialisations were published by fence_mbar_init above, and a releasing arrival
    // costs the 800 clocks of a cluster-wide memory fence)
    if (CL) asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");
    // Let the next kernel in the stream start its own prologue and weight prefetch; everything below
    // that reads or writes memory another kernel may have written comes after griddepcontrol.wait.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    if (warp == kDecWarps) {
        // ------------------------------------------------ producer warp
        const uint32_t unit_tx = (uint32_t)dec_unit_bytes(SG, sym);
        auto issue_weights = [&](const DecStageIter& it, unsigned char* st, uint64_t* bar, int gc) {
            bulk_g2s(st, p.Wq + (size_t)it.u * kBlockWords, (uint32_t)(gc * kBlockBytes), bar);
            bulk_g2s(st + kDecStageS, p.S + (size_t)it.u * (SG * kSBlockHalves), (uint32_t)(gc * SG * kSBlockHalves * 2), bar);
            if (!sym)
                bulk_g2s(st + kStageZ, p.Z + (size_t)it.u * (SG * kZBlockWords), (uint32_t)(gc * SG * kZBlockWords * 4), bar);
        };
        auto issue_rows = [&](const DecStageIter& it, unsigned char* st, int slot_i, uint64_t* bar, int gc) {
            const int g = it.group();  // the stage's units are blocks g .. g + gc - 1 of tile t
            if (a_box) {
                // (always the whole box: chunks past the stage's units are not read, chunks past K are zero)
                if (lane == 0)
                    asm volatile(
                        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                        ::"r"(a_slot0 + (uint32_t)slot_i * a_step), "l"(&tmap_a), "r"(0), "r"(m0), "r"(2 * g), "r"(smem_u32(bar))
                        : "memory");
                return;
            }
            for (int m = lane; m < rows; m += 32) {
                bulk_g2s(st + kStageA + m * kDecARowBytes, p.A + (size_t)(m0 + m) * p.K + (size_t)g * kGroup,
                         (uint32_t)(gc * kGroup * 2), bar);
            }
        };
        auto rows_tx = [&](int gc) -> uint32_t { return a_box ? kABoxBytes : (uint32_t)(rows * gc * (kGroup * 2)); };
        if (a_box && lane == 0) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_a) : "memory");
        // 1. packed weights of the first ring-full of stages: they do not depend on the previous kernel
        const DecStageIter first(p);
        {
            DecStageIter pre(first);
            for (int i = 0; i < p.prefetch && pre.valid(); ++i, pre.next()) {
                if (lane == 0) {
                    const int gc = pre.units();
                    asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(&full[i])),
                                 "r"((uint32_t)gc * unit_tx)
                                 : "memory");
                    issue_weights(pre, stage0 + (size_t)i * stage_bytes, &full[i], gc);
                }
            }
        }
        // 2. the activations may be the previous kernel's output
        asm volatile("griddepcontrol.wait;" ::: "memory");
        int slot = 0, n = 0;
        uint32_t phase = 0;
        for (DecStageIter it(first); it.valid(); it.next(), ++n) {
            const int gc = it.units();
            unsigned char* st = stage0 + (size_t)slot * stage_bytes;
            if (n < p.prefetch) {
                if (lane == 0) mbar_expect_tx(&full[slot], rows_tx(gc));
                __syncwarp();
                issue_rows(it, st, slot, &full[slot], gc);
            } else if (n < stages) {
                // first use of this slot, weights not requested yet: nothing to wait for; the (small) row
                // copies go in front of the weights
                if (lane == 0) mbar_expect_tx(&full[slot], (uint32_t)gc * unit_tx + rows_tx(gc));
                __syncwarp();
                issue_rows(it, st, slot, &full[slot], gc);
                __syncwarp();
                if (lane == 0) issue_weights(it, st, &full[slot], gc);
            } else {
                if (!mbar_wait_producer(&empty[slot], phase ^ 1u)) return;  // status recorded
                if (lane == 0) {
                    mbar_expect_tx(&full[slot], (uint32_t)gc * unit_tx + rows_tx(gc));
                    issue_weights(it, st, &full[slot], gc);
                }
                __syncwarp();
                issue_rows(it, st, slot, &full[slot], gc);
            }
            if (++slot == stages) {
                slot = 0;
                phase ^= 1u;
            }
        }
        if (CL) asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");   // (pairs with the arrival)
        return;
    }

    // ---------------------------------------------------- consumer warps
    const int gq = lane >> 2, tig = lane & 3;
    const int us = warp >> 1;         // which unit of the stage
    const int hh = warp & 1;          // which 32-column half of the tile: 16-column sub-tiles 2 hh, 2 hh + 1
    const int r0 = hh * 2;
    float acc[2][MB][4];
#pragma unroll
    for (int r = 0; r < 2; ++r)
#pragma unroll
        for (int mb = 0; mb < MB; ++mb)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[r][mb][i] = 0.f;

    // Per-thread byte offsets inside a stage (everything else below is an immediate):
    //   weights: this lane's 8 bytes of a column's 64-k line pair, k = 16 tig .. 16 tig + 15, of sub-tile 2 hh
    //   activations: batch row gq, k = 16 tig ..
    //   scales / zeros: the lane's four columns 32 hh + gq, + 8, + 16, + 24 are neighbours (sz_perm)
    const uint32_t stage0_addr = smem_u32(stage0);
    const uint32_t w_off = (uint32_t)(us * kBlockBytes + hh * 1024 + (tig >> 1) * 128 + ((gq + 4 * (tig >> 1)) & 7) * 16 + (tig & 1) * 8);
    // (a stage holds only the `rows` batch rows this CTA has: lanes of absent rows read the last present one,
    // and what they compute lands in output columns that are never stored)
    // -- relative to the slot's activation rows; the 64 k of the unit's second half lie kADc further.
    // Tensor-copy layout: [chunk of 64 k][row][128 B], the 16-byte pieces of a row exchanged by the 128-byte
    // swizzle (piece j of row r at j ^ (r & 7)): the lane's second 16 bytes are at its first address ^ 16.
    const int piece = (2 * tig) ^ gq;
    const uint32_t a_off = a_box ? (uint32_t)(us * 2 * (kRows * 128) + gq * 128 + piece * 16)
                                 : (uint32_t)(us * (kGroup * 2) + min(gq, rows - 1) * kDecARowBytes + tig * 32);
    const uint32_t a_off1 = a_box ? a_off + 1024u
                                  : (uint32_t)(us * (kGroup * 2) + min(8 + gq, rows - 1) * kDecARowBytes + tig * 32);
    constexpr int kADc = a_box ? kRows * 128 : 128;
    // SG = 4 (groups of 32 k): the lane's 16 k of a 64-k half lie in row 2 c + tig / 2
    const int jlane = SG == 4 ? (tig >> 1) : 0;
    const uint32_t s_off = (uint32_t)(kDecStageS + (us * SG + jlane) * (kSBlockHalves * 2) + (32 * hh + 4 * gq) * 2);
    const uint32_t z_off = (uint32_t)(kStageZ + (us * SG + jlane) * (kZBlockWords * 4) + 16 * hh + 2 * gq);

    // scale and zero-point constants of the lane's four columns (index 2 r + b: sub-tile r, column + 8 b)
    uint32_t s2[4], zlo[4], zhi[4];
    auto load_consts = [&](uint32_t st_addr, int j) {
        const uint2 sv = (j == 0)   ? lds64<0>(st_addr + s_off)
                         : (j == 1) ? lds64<kSBlockHalves * 2>(st_addr + s_off)
                                    : lds64<2 * kSBlockHalves * 2>(st_addr + s_off);
        s2[0] = __byte_perm(sv.x, 0, 0x1010);
        s2[1] = __byte_perm(sv.x, 0, 0x3232);
        s2[2] = __byte_perm(sv.y, 0, 0x1010);
        s2[3] = __byte_perm(sv.y, 0, 0x3232);
        if (sym) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                zlo[i] = zconst_lo<BF>(kSymZero);
                zhi[i] = zconst_hi<BF>(kSymZero);
            }
        } else {
            const uint32_t zz = (j == 0)   ? lds16<0>(st_addr + z_off)
                                : (j == 1) ? lds16<kZBlockWords * 4>(st_addr + z_off)
                                           : lds16<2 * kZBlockWords * 4>(st_addr + z_off);
            const uint32_t t = zz * 0x00010001u;     // the four nibbles in both halves
            const uint32_t t4 = t >> 4, t8 = t >> 8, t12 = t >> 12;
            if constexpr (BF) {
                zlo[0] = lop3<kLutAndOr>(t, kMaskLo, kMagicBf);
                zlo[1] = lop3<kLutAndOr>(t4, kMaskLo, kMagicBf);
                zlo[2] = lop3<kLutAndOr>(t8, kMaskLo, kMagicBf);
                zlo[3] = lop3<kLutAndOr>(t12, kMaskLo, kMagicBf);
#pragma unroll
                for (int i = 0; i < 4; ++i) zhi[i] = 0u;
            } else {
                zlo[0] = lop3<kLutAndOr>(t, kMaskLo, kMagicLo);
                zlo[1] = lop3<kLutAndOr>(t4, kMaskLo, kMagicLo);
                zlo[2] = lop3<kLutAndOr>(t8, kMaskLo, kMagicLo);
                zlo[3] = lop3<kLutAndOr>(t12, kMaskLo, kMagicLo);
                zhi[0] = lop3<kLutAndOr>(t << 4, kMaskHi, kMagicHi);
                zhi[1] = lop3<kLutAndOr>(t, kMaskHi, kMagicHi);
                zhi[2] = lop3<kLutAndOr>(t4, kMaskHi, kMagicHi);
                zhi[3] = lop3<kLutAndOr>(t8, kMaskHi, kMagicHi);
            }
        }
    };

    asm volatile("griddepcontrol.wait;" ::: "memory");
    float* const ws_mz = p.ws + (size_t)mz * (2 * (size_t)p.nchunks) * (kRows * kTileN);
    int* const tickets_mz = p.tickets + (size_t)mz * p.T;

    int slot = 0;
    uint32_t phase = 0;
    uint32_t st_addr = stage0_addr;
    uint32_t sa_addr = a_slot0;
    for (int ci = blockIdx.x; ci < p.nchunks; ci += gridDim.x) {
        const int u0 = chunk_begin(p, ci);
        const int u1 = chunk_begin(p, ci + 1);
        if (u0 >= u1) continue;
        int u = u0;
        int t = fast_div(u, p.div_G);
        int tile_end = (t + 1) * p.G;
        int seg_start = u0;
        while (u < u1) {
            const int gc = min(kDecUnitsPerStage, min(u1, tile_end) - u);
            if (!mbar_wait(&full[slot], phase)) return;  // status recorded; every consumer warp sees it
            if (us < gc) {
                const uint32_t wa = st_addr + w_off, aa = sa_addr + a_off, aa1 = sa_addr + a_off1;
                if constexpr (SG == 1) load_consts(st_addr, 0);
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    if constexpr (SG == 2) load_consts(st_addr, c);
                    if constexpr (SG == 4) load_consts(st_addr, 2 * c);
                    // B fragments: batch row 8 mb + gq, 16 consecutive k per lane
                    uint32_t bw[MB][8];
#pragma unroll
                    for (int mb = 0; mb < MB; ++mb) {
                        uint4 x, y;
                        const uint32_t ab = mb == 0 ? aa : aa1;
                        if constexpr (a_box) {
                            if (c == 0) {
                                x = lds128<0>(ab);
                                y = lds128<0>(ab ^ 16u);
                            } else {
                                x = lds128<kADc>(ab);
                                y = lds128<kADc>(ab ^ 16u);
                            }
                        } else if (c == 0) {
                            x = lds128<0>(ab);
                            y = lds128<16>(ab);
                        } else {
                            x = lds128<128>(ab);
                            y = lds128<128 + 16>(ab);
                        }
                        bw[mb][0] = x.x; bw[mb][1] = x.y; bw[mb][2] = x.z; bw[mb][3] = x.w;
                        bw[mb][4] = y.x; bw[mb][5] = y.y; bw[mb][6] = y.z; bw[mb][7] = y.w;
                    }
#pragma unroll
                    for (int r = 0; r < 2; ++r) {
                        // sub-block (c, 2 (2 hh + r)) holds columns 16 rr + gq, the next one columns + 8
                        uint2 va, vb;
                        if (c == 0 && r == 0) { va = lds64<0>(wa); vb = lds64<256>(wa); }
                        else if (c == 0)      { va = lds64<512>(wa); vb = lds64<512 + 256>(wa); }
                        else if (r == 0)      { va = lds64<2048>(wa); vb = lds64<2048 + 256>(wa); }
                        else                  { va = lds64<2048 + 512>(wa); vb = lds64<2048 + 512 + 256>(wa); }
                        const uint32_t wwa[2] = {va.x, va.y}, wwb[2] = {vb.x, vb.y};
#pragma unroll
                        for (int wi = 0; wi < 2; ++wi) {
                            const Pack8 fa = dequant_word<BF>(wwa[wi], zlo[2 * r], zhi[2 * r], s2[2 * r]);
                            const Pack8 fb = dequant_word<BF>(wwb[wi], zlo[2 * r + 1], zhi[2 * r + 1], s2[2 * r + 1]);
#pragma unroll
                            for (int mb = 0; mb < MB; ++mb) {
                                mma_m16n8k16<BF>(acc[r][mb], fa.h[0], fb.h[0], fa.h[1], fb.h[1], bw[mb][4 * wi],
                                                 bw[mb][4 * wi + 1]);
                                mma_m16n8k16<BF>(acc[r][mb], fa.h[2], fb.h[2], fa.h[3], fb.h[3], bw[mb][4 * wi + 2],
                                                 bw[mb][4 * wi + 3]);
                            }
                        }
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[slot]);
            st_addr += (uint32_t)stage_bytes;
            sa_addr += a_step;
            if (++slot == stages) {
                slot = 0;
                phase ^= 1u;
                st_addr = stage0_addr;
                sa_addr = a_slot0;
            }
            u += gc;
            if (u != tile_end && u != u1) continue;

            // ------------------------------------------------ leave tile t: units [seg_start, u)
            consumer_bar();
#pragma unroll
            for (int r = 0; r < 2; ++r)
#pragma unroll
                for (int mb = 0; mb < MB; ++mb)
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int n = (r0 + r) * 16 + gq + (i >= 2 ? 8 : 0);
                        const int m = mb * 8 + 2 * tig + (i & 1);
                        red[(us * kRows + m) * kDecRedStride + n] = acc[r][mb][i];
                        acc[r][mb][i] = 0.f;
                    }
            consumer_bar();
            const int tile_u0 = t * p.G;
            const bool whole = (seg_start == tile_u0) && (u == tile_end);
            // first segment of a chunk -> slot 2 ci, a chunk's continuation into a later tile -> 2 ci + 1
            float* my_slot = ws_mz + (size_t)(2 * ci + (seg_start == u0 ? 0 : 1)) * (kRows * kTileN);
            if (CL && !whole) {
                // slices 1 .. S - 1 -> slot rank - 1 of the exchange buffer of the cluster's CTA 0, which
                // adds them to its own slice 0 in ascending order
                asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");   // the arrival at kernel start
                uint32_t rank;
                asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
                if (rank != 0) {
                    uint32_t xch0, xbar0;
                    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(xch0) : "r"(smem_u32(xch)), "r"(0u));
                    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(xbar0) : "r"(smem_u32(xbar)), "r"(0u));
                    for (int idx = threadIdx.x; idx < rows * kTileN; idx += kDecConsumers) {
                        const int n = idx & (kTileN - 1), m = idx >> 6;
                        float v = red[m * kDecRedStride + n];
#pragma unroll
                        for (int w = 1; w < kDecUnitsPerStage; ++w) v += red[(w * kRows + m) * kDecRedStride + n];
                        asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(xch0 + ((rank - 1u) * (kRows * kTileN) + idx) * 4u),
                                     "f"(v)
                                     : "memory");
                    }
                    // the warp's stores, then one release-arrival per warp on CTA 0's barrier
                    __syncwarp();
                    if (lane == 0)
                        asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(xbar0) : "memory");
                } else {
                    if (!mbar_wait_cluster(xbar, 0u)) return;   // status recorded
                    for (int idx = threadIdx.x; idx < rows * kTileN; idx += kDecConsumers) {
                        const int n = idx & (kTileN - 1), m = idx >> 6;
                        float v = red[m * kDecRedStride + n];
#pragma unroll
                        for (int w = 1; w < kDecUnitsPerStage; ++w) v += red[(w * kRows + m) * kDecRedStride + n];
                        for (int sl = 1; sl < p.split_k; ++sl) v += xch[(sl - 1) * (kRows * kTileN) + idx];
                        p.C[(size_t)(m0 + m) * p.N + (size_t)t * kTileN + n] = finish<BF>(v, t * kTileN + n, p.epi);
                    }
                }
                return;   // one slice per CTA: nothing follows
            }
            for (int idx = threadIdx.x; idx < rows * kTileN; idx += kDecConsumers) {
                const int n = idx & (kTileN - 1), m = idx >> 6;
                float v = red[m * kDecRedStride + n];
#pragma unroll
                for (int w = 1; w < kDecUnitsPerStage; ++w) v += red[(w * kRows + m) * kDecRedStride + n];
                if (whole)
                    p.C[(size_t)(m0 + m) * p.N + (size_t)t * kTileN + n] = finish<BF>(v, t * kTileN + n, p.epi);
                else
                    my_slot[idx] = v;
            }
            if (!whole) {
                __threadfence();  // this thread's partial stores are visible device-wide before the ticket
                consumer_bar();
                const int c_first = chunk_of(p, tile_u0);
                const int c_last = chunk_of(p, tile_end - 1);
                if (threadIdx.x == 0) {
                    const int old = atomicAdd(&tickets_mz[t], 1);
                    const int last = (old == c_last - c_first);
                    if (last) tickets_mz[t] = 0;  // all contributors have arrived: zero for the next call
                    *last_flag = last;
                }
                consumer_bar();
                if (*last_flag) {
                    __threadfence();
                    // contributors in ascending K: chunk c_first (its first segment if it starts at the
                    // tile's first unit, else its continuation), then the first segments of the others
                    const int first_slot = 2 * c_first + (chunk_begin(p, c_first) == tile_u0 ? 0 : 1);
                    for (int idx = threadIdx.x; idx < rows * kTileN; idx += kDecConsumers) {
                        const int n = idx & (kTileN - 1), m = idx >> 6;
                        float v = __ldcg(ws_mz + (size_t)first_slot * (kRows * kTileN) + idx);
                        // four loads in flight at a time (a load per round trip would make the tail
                        // S - 1 trips long); the additions keep the ascending order
                        const float* src = ws_mz + idx;
                        const size_t cstride = (size_t)2 * (kRows * kTileN);
                        int c = c_first + 1;
                        for (; c + 3 <= c_last; c += 4) {
                            const float x0 = __ldcg(src + (size_t)c * cstride), x1 = __ldcg(src + (size_t)(c + 1) * cstride);
                            const float x2 = __ldcg(src + (size_t)(c + 2) * cstride), x3 = __ldcg(src + (size_t)(c + 3) * cstride);
                            v += x0; v += x1; v += x2; v += x3;
                        }
                        if (c + 1 <= c_last) {
                            const float x0 = __ldcg(src + (size_t)c * cstride), x1 = __ldcg(src + (size_t)(c + 1) * cstride);
                            v += x0; v += x1;
                            c += 2;
                        }
                        if (c <= c_last) v += __ldcg(src + (size_t)c * cstride);
                        p.C[(size_t)(m0 + m) * p.N + (size_t)t * kTileN + n] = finish<BF>(v, t * kTileN + n, p.epi);
                    }
                }
            }
            seg_start = u;
            if (u == tile_end) {
                ++t;
                tile_end += p.G;
            }
        }
    }
}

}  // namespace w4a16
