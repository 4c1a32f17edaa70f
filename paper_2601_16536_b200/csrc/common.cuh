// Shared device helpers: packed-layout constants, the device status word, PTX wrappers
// (mbarrier, TMA bulk copy, lop3) used by every kernel of the library.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <stdint.h>

namespace w4a16 {

// ---------------------------------------------------------------------------------
// Packed layout.  The weight matrix is cut into blocks of NT = 64 columns (n) by one
// quantization group (128 k).  Block (t, g), t = n / 64, g = k / 128, G = K / 128, sits at
// position t*G + g of each packed buffer, so a K-slice of a column tile is one contiguous
// byte range in each buffer (one TMA bulk copy each).
//
//   Wq  : 1024 uint32 (4 KiB) per block.  Every word holds 8 consecutive k of ONE column n.
//         The block is cut into 16 sub-blocks of 256 B: sub-block (c, rb), c = (k % 128) / 64,
//         rb = (n % 64) / 8, at byte (c*8 + rb)*256, holds columns 8rb .. 8rb+7 (rho = n % 8)
//         times 64 k as two 128-byte lines, line i = (k % 64) / 32.  Column rho's 16 bytes of
//         line i (four words w = 0..3, k = 64c + 32i + 8w .. +7) sit at slot (rho + 4i) % 8 of
//         the line.  With that rotation
//           - eight threads that each own one column read their 16-byte chunk of a line from
//             eight different slots (one 128-byte wavefront), and
//           - a warp whose lane (gq = lane / 4, tig = lane % 4) reads 8 bytes of column gq at
//             k = 16 tig .. 16 tig + 15 touches every bank once per half-warp.
//         Inside a word, nibble p holds k offset 2 (p % 4) + p / 4, i.e. nibbles 0,4 = k+0,k+1;
//         1,5 = k+2,k+3; 2,6 = k+4,k+5; 3,7 = k+6,k+7: the masks 0x000f000f / 0x00f000f0 on the
//         word and on the word >> 8 then give four FP16x2 registers in ascending k.
//   S   : per block, one row of 64 16-bit scales (FP16 or BF16 bit patterns) per quantization group
//         inside the block: sg = 128 / group rows (group = 128, 64 or 32), row j = (k % 128) / group.
//         Inside a row the scale of column c = n % 64 sits at position sz_perm(c): the four columns
//         32 h + gq, + 8, + 16, + 24 that one lane of the warp-MMA kernel owns are neighbours (one
//         64-bit shared load fetches the lane's four scales).
//   Z   : the same rows and the same permutation, 4 bits per zero point (8 uint32 per row).  A
//         symmetric format (zero point 8 for every weight) has no Z buffer at all.
// ---------------------------------------------------------------------------------
constexpr int kGroup = 128;        // k per packed block (the scheduling unit); quantization groups divide it
constexpr int kTileN = 64;
constexpr int kBlockWords = 1024;  // uint32 per (tile, k-block) block of Wq
constexpr int kBlockBytes = 4096;
constexpr int kSBlockHalves = 64;  // scales per row (one row per quantization group of the block)
constexpr int kZBlockWords = 8;    // zero-point words per row
constexpr int kSymZero = 8;        // zero point of the symmetric format (Eq. 1 with z fixed: q - 8 in -8 .. 7)

// Position of column c (0..63) inside a row of scales / zero points.
__host__ __device__ constexpr int sz_perm(int c) {
    return (c & 32) + 4 * (c & 7) + 2 * ((c >> 4) & 1) + ((c >> 3) & 1);
}
__host__ __device__ constexpr bool group_ok(int group) { return group == 128 || group == 64 || group == 32; }

// Word index inside a block of the word that holds column `col` (0..63) at k = 8*kw .. 8*kw+7
// (kw = 0..15 inside the group).
__host__ __device__ constexpr int block_word_index(int col, int kw) {
    return ((kw >> 3) * 8 + (col >> 3)) * 64 + ((kw >> 2) & 1) * 32 + (((col & 7) + 4 * ((kw >> 2) & 1)) & 7) * 4 +
           (kw & 3);
}

// Status word: a kernel whose bounded wait runs out ORs a code in here and returns.  One word per
// translation unit of the library (the kernels are compiled in several); w4a16_device_status reads
// and clears all of them through status_take() of each unit.
static __device__ int g_status_word = 0;
constexpr int kStatusMbarTimeout = 1;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // every bounded wait of the GEMM kernels: two seconds

__device__ __forceinline__ void report_status(int code) { atomicOr(&g_status_word, code); }
// Host: read and clear this translation unit's word (the device must be idle); -1 if a CUDA call fails.
static inline int status_take_this_unit() {
    int v = 0, zero = 0;
    if (cudaMemcpyFromSymbol(&v, g_status_word, sizeof(int)) != cudaSuccess ||
        cudaMemcpyToSymbol(g_status_word, &zero, sizeof(int)) != cudaSuccess) {
        cudaGetLastError();
        return -1;
    }
    return v;
}

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Bounded wait: returns false (after recording the status code) if the phase does not complete
// within about two seconds.  Fast path, inlined: one try_wait (about 40 clocks when the phase is
// already complete).  Slow path, a function of its own so that the many waits of a kernel do not
// each carry a copy of the loop: try_wait with a suspend-time hint, so that a waiting warp sleeps in
// the barrier unit instead of spending issue slots on polling, and a wall-clock limit read from
// %globaltimer (the hint is only a hint: an iteration count would not bound the time).
static __device__ __noinline__ bool mbar_wait_slow(uint32_t bar_addr, uint32_t parity, unsigned long long limit_ns) {
    uint32_t ok;
    unsigned long long t0;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    for (;;) {
        asm volatile(
            "{\n\t"
            ".reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t"
            "}"
            : "=r"(ok)
            : "r"(bar_addr), "r"(parity), "r"(20000u)
            : "memory");
        if (ok) return true;
        unsigned long long t1;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
        if (t1 - t0 > limit_ns) break;
    }
    report_status(kStatusMbarTimeout);
    return false;
}
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, unsigned long long limit_ns = kWaitLimitNs) {
    uint32_t ok;
    const uint32_t addr = smem_u32(bar);
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t"
        "}"
        : "=r"(ok)
        : "r"(addr), "r"(parity)
        : "memory");
    if (ok) return true;
    return mbar_wait_slow(addr, parity, limit_ns);
}

// The same bounded wait with cluster-scope acquire: for a barrier that CTAs of the cluster arrive on
// after writing this CTA's shared memory.
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    unsigned long long t0;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    for (;;) {
        asm volatile(
            "{\n\t"
            ".reg .pred p;\n\t"
            "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2, %3;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t"
            "}"
            : "=r"(ok)
            : "r"(smem_u32(bar)), "r"(parity), "r"(20000u)
            : "memory");
        if (ok) return true;
        unsigned long long t1;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
        if (t1 - t0 > kWaitLimitNs) break;
    }
    report_status(kStatusMbarTimeout);
    return false;
}

// One lane of a converged warp (warp-uniform control flow keeps addresses and descriptors in
// uniform registers; only the issuing instruction itself is predicated on the elected lane).
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(pred));
    return pred != 0;
}

// TMA bulk copy global -> shared (1-D, no tensor map).  Addresses and size are multiples
// of 16 bytes.  Completion is signalled on `bar` as transaction bytes.
__device__ __forceinline__ void bulk_g2s(void* smem_dst, const void* gmem_src, uint32_t bytes, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
            smem_u32(smem_dst)),
        "l"(gmem_src), "r"(bytes), "r"(smem_u32(bar))
        : "memory");
}

// n / d for 0 <= n < 2^31 as a multiplication and a shift: the chunk arithmetic of the kernels stands at the head of
// every CTA's critical path (the producer warp cannot request anything before it knows its first unit), and
// a hardware-less 32-bit division costs about 100 clocks of dependent instructions, a 64-bit one several
// hundred.  shift = 31 + ceil(log2 d), mul = ceil(2^shift / d) < 2^32 gives the exact quotient.
struct FastDiv {
    uint32_t mul, shift;
};
inline FastDiv fast_div_make(uint32_t d) {
    uint32_t c = 0;
    while ((1ull << c) < d) ++c;
    FastDiv f;
    f.shift = 31 + c;
    f.mul = (uint32_t)(((1ull << f.shift) + d - 1) / d);
    return f;
}
__device__ __forceinline__ int fast_div(int n, FastDiv f) {
    return (int)(((unsigned long long)(uint32_t)n * f.mul) >> f.shift);
}

// Tiled tensor copies (TMA) global -> shared; completion as transaction bytes on an mbarrier.
__device__ __forceinline__ void tma_load_2d(void* smem_dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(smem_dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar))
        : "memory");
}
__device__ __forceinline__ void tma_load_3d(void* smem_dst, const CUtensorMap* map, int x, int y, int z, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(smem_u32(smem_dst)), "l"(map), "r"(x), "r"(y), "r"(z), "r"(smem_u32(bar))
        : "memory");
}

template <int kLut>
__device__ __forceinline__ uint32_t lop3(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t r;
    asm("lop3.b32 %0, %1, %2, %3, %4;" : "=r"(r) : "r"(a), "r"(b), "r"(c), "n"(kLut));
    return r;
}

// ------------------------------------------------------------------ nibble -> FP16 / BF16
// Everything below works on 32-bit registers that hold two 16-bit floating-point values; the
// template parameter BF selects BF16 (true) or FP16 (false) arithmetic.
//
// FP16 (ten fraction bits):
//   (w & 0x000f000f) | 0x64006400 = (1024 + q_a, 1024 + q_b) for the nibbles at bits 0..3 / 16..19;
//   (w & 0x00f000f0) | 0x54005400 = (  64 + q_a,   64 + q_b) for the nibbles at bits 4..7 / 20..23
//   (the spacing of FP16 values at 64 is 1/16, so a nibble four bits up counts in units of one).
//   Subtracting (1024 + z) resp. (64 + z) gives q - z exactly.
// BF16 (seven fraction bits): a nibble fits the fraction only at bits 0..3, so the word is shifted by
//   0, 4, 8, 12;  (w' & 0x000f000f) | 0x43004300 = (128 + q_a, 128 + q_b);  minus (128 + z) is exact.
// Then ONE multiply by the scale in the same format: w16 = rn((q - z) * s), the single rounding of
// Algorithm 1's "Dequantize to FP16" (resp. BF16).
constexpr uint32_t kMaskLo = 0x000f000fu;
constexpr uint32_t kMaskHi = 0x00f000f0u;
constexpr uint32_t kMagicLo = 0x64006400u;   // FP16 1024.0 twice
constexpr uint32_t kMagicHi = 0x54005400u;   // FP16 64.0 twice
constexpr uint32_t kMagicBf = 0x43004300u;   // BF16 128.0 twice
constexpr int kLutAndOr = (0xF0 & 0xCC) | 0xAA;  // (a & b) | c

template <bool BF>
__device__ __forceinline__ uint32_t sub2(uint32_t a, uint32_t b) {
    uint32_t r;
    if constexpr (BF) asm("sub.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    else asm("sub.f16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}
template <bool BF>
__device__ __forceinline__ uint32_t mul2(uint32_t a, uint32_t b) {
    uint32_t r;
    if constexpr (BF) asm("mul.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    else asm("mul.f16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

// The two per-column constants of the exact subtraction, both halves alike.
//   FP16: lo = 1024 + z, hi = 64 + z;  BF16: lo = 128 + z (hi unused).
template <bool BF>
__device__ __forceinline__ uint32_t zconst_lo(uint32_t z) {
    return BF ? (z * 0x00010001u + kMagicBf) : (z * 0x00010001u + kMagicLo);
}
template <bool BF>
__device__ __forceinline__ uint32_t zconst_hi(uint32_t z) {
    return BF ? 0u : (z * 0x00100010u + kMagicHi);
}

// Eight weights of one column, ascending k, as four register pairs: h[j] = (k + 2j, k + 2j + 1).
struct Pack8 {
    uint32_t h[4];
};

// One packed word -> exact (q - z) for its eight k.
template <bool BF>
__device__ __forceinline__ Pack8 unpack_word(uint32_t w, uint32_t zlo, uint32_t zhi) {
    Pack8 f;
    if constexpr (BF) {
        f.h[0] = sub2<true>(lop3<kLutAndOr>(w, kMaskLo, kMagicBf), zlo);
        f.h[1] = sub2<true>(lop3<kLutAndOr>(w >> 4, kMaskLo, kMagicBf), zlo);
        f.h[2] = sub2<true>(lop3<kLutAndOr>(w >> 8, kMaskLo, kMagicBf), zlo);
        f.h[3] = sub2<true>(lop3<kLutAndOr>(w >> 12, kMaskLo, kMagicBf), zlo);
    } else {
        const uint32_t w8 = w >> 8;
        f.h[0] = sub2<false>(lop3<kLutAndOr>(w, kMaskLo, kMagicLo), zlo);
        f.h[1] = sub2<false>(lop3<kLutAndOr>(w, kMaskHi, kMagicHi), zhi);
        f.h[2] = sub2<false>(lop3<kLutAndOr>(w8, kMaskLo, kMagicLo), zlo);
        f.h[3] = sub2<false>(lop3<kLutAndOr>(w8, kMaskHi, kMagicHi), zhi);
    }
    return f;
}

// One packed word -> w16 = rn((q - z) * s) for its eight k (s2 = the column's scale in both halves).
// Every kernel that feeds tensor cores goes through here: the multiplicand of the GEMM is the
// weight rounded to the 16-bit format, as in Algorithm 1, Phase 1.
template <bool BF>
__device__ __forceinline__ Pack8 dequant_word(uint32_t w, uint32_t zlo, uint32_t zhi, uint32_t s2) {
    Pack8 f = unpack_word<BF>(w, zlo, zhi);
#pragma unroll
    for (int j = 0; j < 4; ++j) f.h[j] = mul2<BF>(f.h[j], s2);
    return f;
}

// FP32 -> 16-bit output, round to nearest even (the one cast of Algorithm 1, Phase 3).
template <bool BF>
__device__ __forceinline__ uint16_t cast_out(float v) {
    uint16_t r;
    if constexpr (BF) asm("cvt.rn.bf16.f32 %0, %1;" : "=h"(r) : "f"(v));
    else asm("cvt.rn.f16.f32 %0, %1;" : "=h"(r) : "f"(v));
    return r;
}
// Optional work fused into the final cast (none of it is in the paper's Algorithm 1; it stands for the
// step that follows a linear layer): y = act(acc + bias[n]) in FP32, then the one rounding to 16 bits.
constexpr int kActNone = 0, kActRelu = 1, kActSilu = 2;
struct Epilogue {
    const uint16_t* bias;   // [N] in the output's 16-bit format, or nullptr
    int act;                // kActNone / kActRelu / kActSilu
};

// 16-bit value -> FP32 (exact).
template <bool BF>
__device__ __forceinline__ float widen(uint16_t v) {
    if constexpr (BF) return __uint_as_float((uint32_t)v << 16);
    float r;
    asm("cvt.f32.f16 %0, %1;" : "=f"(r) : "h"(v));
    return r;
}

// The final value of C[m, n] from its FP32 sum.
template <bool BF>
__device__ __forceinline__ uint16_t finish(float v, int n, const Epilogue& e) {
    if (e.bias != nullptr) v += widen<BF>(e.bias[n]);
    if (e.act == kActRelu) v = fmaxf(v, 0.f);
    else if (e.act == kActSilu) v = v / (1.f + __expf(-v));
    return cast_out<BF>(v);
}

}  // namespace w4a16
