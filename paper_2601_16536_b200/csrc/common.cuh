// Shared device helpers: packed-layout constants, the device status word, PTX wrappers
// (mbarrier, TMA bulk copy, lop3) used by every kernel of the library.
#pragma once

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
//   S   : 64 FP16 per block, element n % 64.
//   Z   : 8 uint32 per block, word (n % 64) / 8, nibble n % 8.
// ---------------------------------------------------------------------------------
constexpr int kGroup = 128;
constexpr int kTileN = 64;
constexpr int kBlockWords = 1024;  // uint32 per (tile, group) block of Wq
constexpr int kBlockBytes = 4096;
constexpr int kSBlockHalves = 64;
constexpr int kZBlockWords = 8;

// Word index inside a block of the word that holds column `col` (0..63) at k = 8*kw .. 8*kw+7
// (kw = 0..15 inside the group).
__host__ __device__ constexpr int block_word_index(int col, int kw) {
    return ((kw >> 3) * 8 + (col >> 3)) * 64 + ((kw >> 2) & 1) * 32 + (((col & 7) + 4 * ((kw >> 2) & 1)) & 7) * 4 +
           (kw & 3);
}

// Status word: a kernel whose bounded wait runs out ORs a code in here and returns.
__device__ int g_status_word = 0;
constexpr int kStatusMbarTimeout = 1;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // every bounded wait of the GEMM kernels: two seconds

__device__ __forceinline__ void report_status(int code) { atomicOr(&g_status_word, code); }

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
// within about two seconds.  Fast path: one try_wait (about 40 clocks when the phase is already
// complete).  Slow path: try_wait with a suspend-time hint, so that a waiting warp sleeps in the
// barrier unit instead of spending issue slots on polling, and a wall-clock limit read from
// %globaltimer (the hint is only a hint: an iteration count would not bound the time).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, unsigned long long limit_ns = kWaitLimitNs) {
    uint32_t ok;
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t"
        "}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    if (ok) return true;
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
            : "r"(smem_u32(bar)), "r"(parity), "r"(20000u)
            : "memory");
        if (ok) return true;
        unsigned long long t1;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
        if (t1 - t0 > limit_ns) break;
    }
    report_status(kStatusMbarTimeout);
    return false;
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

template <int kLut>
__device__ __forceinline__ uint32_t lop3(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t r;
    asm("lop3.b32 %0, %1, %2, %3, %4;" : "=r"(r) : "r"(a), "r"(b), "r"(c), "n"(kLut));
    return r;
}

// ------------------------------------------------------------------ nibble -> FP16
// (w & 0x000f000f) | 0x64006400 is the FP16 pair (1024 + q_a, 1024 + q_b) for the nibbles
// at bits 0..3 and 16..19;  (w & 0x00f000f0) | 0x64006400 is (1024 + 16 q_a, 1024 + 16 q_b)
// for the nibbles at bits 4..7 and 20..23.  Both are exact FP16 values, so
//   lo - (1024 + z)            = q - z   exactly (FP16 subtract of nearby integers)
//   hi * (1/16) - (64 + z)     = q - z   exactly (FMA, the exact result is representable)
constexpr uint32_t kMaskLo = 0x000f000fu;
constexpr uint32_t kMaskHi = 0x00f000f0u;
constexpr uint32_t kMagic = 0x64006400u;  // FP16 1024.0 in both halves
constexpr int kLutAndOr = (0xF0 & 0xCC) | 0xAA;  // (a & b) | c

// Eight weights of one column, ascending k, as four FP16 pairs.
struct Half8 {
    __half2 h[4];  // h[j] = (k + 2j, k + 2j + 1)
};

__device__ __forceinline__ __half2 u32_as_h2(uint32_t v) {
    return *reinterpret_cast<__half2*>(&v);
}
__device__ __forceinline__ uint32_t h2_as_u32(__half2 v) {
    return *reinterpret_cast<uint32_t*>(&v);
}

// zlo = FP16x2 (1024 + z) in both halves; zhi = FP16x2 -(64 + z) in both halves.
__device__ __forceinline__ uint32_t zmagic_lo(uint32_t z) { return z * 0x00010001u + kMagic; }
__device__ __forceinline__ uint32_t zmagic_hi(uint32_t z) { return z * 0x00100010u + 0xD400D400u; }

// One packed word -> exact (q - z) for its eight k.
__device__ __forceinline__ Half8 unpack_word(uint32_t w, __half2 zlo, __half2 zhi) {
    const __half2 sixteenth = __float2half2_rn(0.0625f);
    Half8 f;
    const uint32_t w8 = w >> 8;
    f.h[0] = __hsub2(u32_as_h2(lop3<kLutAndOr>(w, kMaskLo, kMagic)), zlo);
    f.h[1] = __hfma2(u32_as_h2(lop3<kLutAndOr>(w, kMaskHi, kMagic)), sixteenth, zhi);
    f.h[2] = __hsub2(u32_as_h2(lop3<kLutAndOr>(w8, kMaskLo, kMagic)), zlo);
    f.h[3] = __hfma2(u32_as_h2(lop3<kLutAndOr>(w8, kMaskHi, kMagic)), sixteenth, zhi);
    return f;
}

// One packed word -> w16 = fp16_rn((q - z) * s) for its eight k: exact (q - z), then one FP16
// multiply by the column's scale (both halves of s2).  This is Algorithm 1's "Dequantize to
// FP16": the multiplicand of the GEMM is the FP16-rounded weight, so every kernel that feeds
// tensor cores goes through here.
__device__ __forceinline__ Half8 dequant_word(uint32_t w, __half2 zlo, __half2 zhi, __half2 s2) {
    Half8 f = unpack_word(w, zlo, zhi);
#pragma unroll
    for (int j = 0; j < 4; ++j) f.h[j] = __hmul2(f.h[j], s2);
    return f;
}

}  // namespace w4a16
