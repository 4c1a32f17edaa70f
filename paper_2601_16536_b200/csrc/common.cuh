// Shared device helpers: packed-layout constants, the device status word, PTX wrappers
// (mbarrier, TMA bulk copy, lop3) used by every kernel of the library.
#pragma once

#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <stdint.h>

namespace w4a16 {

// ---------------------------------------------------------------------------------
// Packed layout.  The weight matrix is cut into blocks of NT = 64 columns (n) by one
// quantization group (128 k).  Block (t, g), t = n / 64, g = k / 128, G = K / 128:
//
//   Wq  : 1024 uint32 (4 KiB) at word offset (t*G + g) * 1024, index
//           ((c*4 + r)*32 + lane)*4 + j
//         c = (k % 128) / 64  (64-wide k chunk), r = (n % 64) / 16 (16-row sub-tile),
//         lane = gq*4 + tig (gq = 0..7, tig = 0..3), j = 0..3.
//         The word holds 8 nibbles of rows n_lo = 64t + 16r + gq and n_hi = n_lo + 8 at
//         k0 = 128g + 64c + 16 tig + 4j:
//           nibble 0: (n_lo, k0)    nibble 4: (n_lo, k0+1)
//           nibble 1: (n_hi, k0)    nibble 5: (n_hi, k0+1)
//           nibble 2: (n_lo, k0+2)  nibble 6: (n_lo, k0+3)
//           nibble 3: (n_hi, k0+2)  nibble 7: (n_hi, k0+3)
//         so that one 128-bit load gives a lane 16 consecutive k of two rows, and the
//         masks 0x000f000f / 0x00f000f0 on the word and on the word >> 8 give the four
//         FP16x2 registers of an m16n8k16 A fragment (rows = n, columns = k).
//   S   : 64 FP16 at element offset (t*G + g) * 64, index gq*8 + r*2 + h  (row 16r+gq+8h)
//   Z   : 8 uint32 at word offset (t*G + g) * 8, word gq, nibble r*2 + h   (same row)
//
// All blocks of one column tile t are contiguous in g, so a K-slice of a tile is one
// contiguous byte range in each of the three buffers (one TMA bulk copy each).
// ---------------------------------------------------------------------------------
constexpr int kGroup = 128;
constexpr int kTileN = 64;
constexpr int kBlockWords = 1024;  // uint32 per (tile, group) block of Wq
constexpr int kBlockBytes = 4096;
constexpr int kSBlockHalves = 64;
constexpr int kZBlockWords = 8;

// Status word: a kernel whose bounded wait runs out ORs a code in here and returns.
__device__ int g_status_word = 0;
constexpr int kStatusMbarTimeout = 1;
constexpr int kStatusTmemAlloc = 2;
constexpr int kStatusTicket = 4;

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
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: returns false (after recording the status code) if the phase never
// completes.  try_wait itself blocks for a hardware-defined slice, so the limit below is
// far beyond any legitimate wait (seconds), yet finite.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
    for (uint32_t it = 0; it < (1u << 22); ++it) {
        if (mbar_try_wait(bar, parity)) return true;
    }
    report_status(kStatusMbarTimeout);
    return false;
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

struct Frag4 {
    __half2 lo_a;  // rows n_lo, k0,   k0+1   (A-fragment register a0)
    __half2 hi_a;  // rows n_hi, k0,   k0+1   (a1)
    __half2 lo_b;  // rows n_lo, k0+2, k0+3   (a2)
    __half2 hi_b;  // rows n_hi, k0+2, k0+3   (a3)
};

__device__ __forceinline__ __half2 u32_as_h2(uint32_t v) {
    return *reinterpret_cast<__half2*>(&v);
}
__device__ __forceinline__ uint32_t h2_as_u32(__half2 v) {
    return *reinterpret_cast<uint32_t*>(&v);
}

// zlo = FP16x2 (1024 + z_lo) in both halves; zhi = FP16x2 -(64 + z_hi) in both halves.
__device__ __forceinline__ uint32_t zmagic_lo(uint32_t z) { return z * 0x00010001u + kMagic; }
__device__ __forceinline__ uint32_t zmagic_hi(uint32_t z) { return z * 0x00100010u + 0xD400D400u; }

// One packed word -> exact (q - z) as four FP16 pairs.
__device__ __forceinline__ Frag4 unpack_word(uint32_t w, __half2 zlo, __half2 zhi) {
    const __half2 sixteenth = __float2half2_rn(0.0625f);
    Frag4 f;
    uint32_t w8 = w >> 8;
    f.lo_a = __hsub2(u32_as_h2(lop3<kLutAndOr>(w, kMaskLo, kMagic)), zlo);
    f.hi_a = __hfma2(u32_as_h2(lop3<kLutAndOr>(w, kMaskHi, kMagic)), sixteenth, zhi);
    f.lo_b = __hsub2(u32_as_h2(lop3<kLutAndOr>(w8, kMaskLo, kMagic)), zlo);
    f.hi_b = __hfma2(u32_as_h2(lop3<kLutAndOr>(w8, kMaskHi, kMagic)), sixteenth, zhi);
    return f;
}

// One packed word -> four FP16 pairs of w16 = fp16_rn((q - z) * s): exact (q - z), then one
// FP16 multiply by the row's scale (both halves of s_lo / s_hi hold the scale of n_lo / n_hi).
// This is Algorithm 1's "Dequantize to FP16": the multiplicand of the GEMM is the FP16-rounded
// weight, so every kernel that feeds tensor cores goes through here.
__device__ __forceinline__ Frag4 dequant_word(uint32_t w, __half2 zlo, __half2 zhi, __half2 s_lo, __half2 s_hi) {
    Frag4 f = unpack_word(w, zlo, zhi);
    f.lo_a = __hmul2(f.lo_a, s_lo);
    f.hi_a = __hmul2(f.hi_a, s_hi);
    f.lo_b = __hmul2(f.lo_b, s_lo);
    f.hi_b = __hmul2(f.hi_b, s_hi);
    return f;
}

}  // namespace w4a16
