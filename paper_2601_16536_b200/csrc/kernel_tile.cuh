// Tensor-core tile kernel of the W4A16 GEMM: tcgen05.mma with the accumulator in tensor memory.
//
// The product is computed transposed, C^T[n, m] = sum_k W16[k, n] A[m, k], so that the
// DEQUANTIZED WEIGHTS are the MMA's 128-row A operand and live only in tensor memory:
//
//   HBM --128-bit loads--> registers (packed nibbles, scale, zero)    16 dequant warps,
//   registers: unpack, (q - z) exact, * s in FP16                      one column n per thread
//   registers --tcgen05.st--> TMEM (A operand, one column n per lane, k packed along columns)
//   HBM --TMA tensor (128B swizzle)--> shared (activation tile, MT rows m x 64 k): B operand
//   tcgen05.mma.kind::f16  D[128 n x MT m] (FP32, TMEM) += A(TMEM) . B(shared)   one elected lane
//   TMEM --tcgen05.ld--> registers -> FP16 C, or FP32 partial tile + ticket (Split-K)
//
// so packed weights go from HBM straight to registers, dequantized weights never touch shared or
// global memory (Algorithm 1's Phase 1 output stays on chip), and the activation tile is re-used
// by all 128 columns of the CTA tile.
//
// Work is counted in units: one unit = 128 columns x one group (128 k) of one batch tile, numbered
// U = (batch tile * NT + column tile) * G + group.  The unit range is cut into chunks, each CTA of
// the persistent grid walks its chunk(s) front to back:
//   - balanced (split_k == 0): as many chunks as CTAs, equal to within one unit; a chunk may start
//     and end inside a tile's K range and may cover several whole tiles in between;
//   - classic Split-K (split_k = S): every tile's K range is cut into S slices of whole groups
//     (Algorithm 1, Phase 2), chunks dealt round-robin.
// The part of a chunk inside one tile is a segment: the accumulator is zeroed at its first MMA and
// drained after its last.  A segment that covers a whole tile is cast to FP16 and stored; any other
// segment leaves as an FP32 partial tile in the workspace, and the warp that draws the last ticket
// of its 32-column x MT/4-row region adds the partial regions in ascending K order (Phase 3).
// No warp ever waits for another CTA, and the order of the sum is fixed, so results are
// bit-identical from run to run.
//
// One pipeline stage is a whole group (128 k, eight MMAs) for batch tiles of up to 64 rows and half
// a group (64 k, four MMAs) above: narrow tiles are bound by per-stage work other than the MMAs
// (the dequant warps' instruction streams, the control warps' loops), wide ones by the tensor pipe.
// A ring of R slots holds, per slot, the stage's activation boxes in shared memory and its
// dequantized weights in tensor memory (32 or 64 columns; six or eight slots fit beside the
// accumulators); the MMAs of a stage release both with one commit.  Four sets of four dequant
// warps take stages round-robin; inside a set warp w owns TMEM lanes 32 (w % 4) .. + 31.  Each
// thread keeps the packed words of its next two or three stages in registers (loads issued that
// far ahead, pointers stepped, no register copies).  Tiles of up to 32 rows have three MMA-issuing
// warps that take the stages round-robin, each summing into an accumulator of its own (the epilogue
// adds them in stage order); the others have one issuer, and two accumulators that alternate
// between segments (MT = 16, 64, 128), so one drains while the next fills.  The packed weights do not depend on the
// previous kernel in the stream: under programmatic dependent launch the dequant warps load and
// convert weights until the TMEM ring is full before anything waits for that kernel; only
// activations, C and the workspace are touched after griddepcontrol.wait.
// The producer and issuer warps run warp-uniform loops and elect one lane per instruction, which
// keeps descriptors in uniform registers.  All waits are bounded mbarrier waits; a wait that runs
// out records a status code and the CTA drains and exits (TMEM is always released).
//
// Which schedule a shape gets when the caller leaves split_k open is the host's choice (api.cu):
// partial tiles are dear (FP32 store, ticket, reload; in mid-chunk they also stall the pipeline), so
// balanced chunks are used only where the SMs left idle by whole slices or whole tiles cost more.
#pragma once


#include "common.cuh"

namespace w4a16 {

constexpr int kTileCols = 128;                      // n per CTA tile = UMMA M
constexpr int kTileBoxK = 64;                       // k per activation TMA box (one 128-byte swizzle row)
// k per pipeline stage: a whole group for narrow batch tiles (twice the MMAs per barrier round: the
// issuing lane and the per-stage synchronisation are what bounds them), half a group otherwise
__host__ __device__ constexpr int tile_stage_k(int mt) { return mt <= 64 ? 128 : 64; }
constexpr int kTileDequantWarps = 16;               // four sets of four (one warp per TMEM lane quarter)
constexpr int kTileSets = kTileDequantWarps / 4;
// MMA-issuing warps.  With narrow batch tiles one issuing warp is busy nearly all the time (a lone
// warp of dependent scalar code beside sixteen busy dequant warps needs 600 to 700 clocks per stage,
// of which the eight MMAs are about 100), so for tiles of up to 32 rows the stages are dealt to three
// issuers, each with an accumulator of its own; the epilogue adds the accumulators in issuer order.
// Measured at K = 11008, N = 4096: 14.0 -> 13.0 us at M = 16; 64-row tiles are faster with one issuer
// and two alternating accumulators (16.9 against 18.3 us), so the split stops at 32 rows.
// An issuer must meet every phase of the `full` barriers it waits on, and a dequant set every phase
// of its `retired` barriers: the ring size has to be an even multiple of the issuer count (host).
__host__ __device__ constexpr int tile_issuers(int mt) { return mt <= 32 ? 3 : 1; }
// producer, issuers, dequant / epilogue warps
__host__ __device__ constexpr int tile_threads(int mt) { return (1 + tile_issuers(mt) + kTileDequantWarps) * 32; }
// accumulators per issuer that alternate between segments, and the TMEM columns between accumulators
__host__ __device__ constexpr int tile_dbufs(int mt) { return mt <= 16 ? 2 : mt <= 32 ? 1 : mt <= 128 ? 2 : 1; }
__host__ __device__ constexpr int tile_d_stride(int mt) { return mt <= 64 ? mt : 128; }
constexpr int kTileMaxStages = 8;                   // ring slots: activation boxes + stage_k / 2 TMEM columns each
// TMEM columns: the accumulators first (two of up to 128 columns, or one of 256), then the operand ring
__host__ __device__ constexpr int tile_a_col_base(int mt) { return mt <= 64 ? 128 : 256; }
__host__ __device__ constexpr int tile_max_slots(int mt) { return (512 - tile_a_col_base(mt)) / (tile_stage_k(mt) / 2); }
// stages of packed words a dequant thread holds in registers (loads issued that far ahead)
__host__ __device__ constexpr int tile_prefetch(int mt) { return mt <= 64 ? 2 : 3; }
constexpr int kTileBarBytes = 1024;

__host__ __device__ constexpr int tile_stage_bytes(int mt) { return mt * tile_stage_k(mt) * 2; }

struct TileParams {
    const uint32_t* Wq;
    const uint16_t* S;
    const uint32_t* Z;   // nullptr: symmetric format, zero point 8
    uint16_t* C;
    float* ws;       // partial tiles: [2 * nchunks slots][MT][128] FP32
    int* tickets;    // zeroed counters: [tile][16 epilogue warps]
    int M, N, K, G;
    int n_tiles;     // NT = ceil(N / 128)
    int m_tiles;     // ceil(M / MT)
    int split_k;     // 0: balanced chunks; S >= 1: classic Split-K
    int nchunks;
    int stages;
    int defer_reduce;   // 1: partial tiles are only stored; tile_splitk_reduce_kernel sums them (classic slices)
    // chunk arithmetic, prepared by the host (tile_fill_chunk_math); units = m_tiles n_tiles G < 2^31
    FastDiv div_G, div_split, div_nchunks, div_ntiles;
    int slice_base, slice_rem;   // classic: G / split_k, G % split_k
    int bal_q, bal_r;            // balanced: units / nchunks, units % nchunks
    Epilogue epi;
};

inline void tile_fill_chunk_math(TileParams& p) {
    p.div_G = fast_div_make((uint32_t)p.G);
    p.div_split = fast_div_make((uint32_t)(p.split_k > 0 ? p.split_k : 1));
    p.div_nchunks = fast_div_make((uint32_t)p.nchunks);
    p.div_ntiles = fast_div_make((uint32_t)p.n_tiles);
    p.slice_base = p.split_k > 0 ? p.G / p.split_k : 0;
    p.slice_rem = p.split_k > 0 ? p.G % p.split_k : 0;
    const long long units = (long long)p.m_tiles * p.n_tiles * p.G;
    p.bal_q = (int)(units / p.nchunks);
    p.bal_r = (int)(units % p.nchunks);
}

// ------------------------------------------------------------------ tcgen05 / TMA wrappers
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
__device__ __forceinline__ void tc_st16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
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
__device__ __forceinline__ void tc_ld8(uint32_t taddr, uint32_t (&r)[8]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr)
                 : "memory");
}
__device__ __forceinline__ void tc_ld4(uint32_t taddr, uint32_t (&r)[4]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
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

// kind::f16 instruction descriptor: FP32 accumulator, A and B both FP16 or both BF16, both K-major,
// M = 128, N = mt.
__host__ __device__ constexpr uint32_t tile_idesc(int mt, bool bf) {
    return (1u << 4) | (bf ? ((1u << 7) | (1u << 10)) : 0u) | ((uint32_t)(mt >> 3) << 17) |
           ((uint32_t)(kTileCols >> 4) << 24);
}

// ------------------------------------------------------------------ chunk schedule
// First unit of chunk i (i == nchunks gives the end of the last chunk).  Multiply-and-shift divisions with the
// host's constants: every role's walk starts here, ahead of its first request, and with real divisions (two of
// them 64-bit) this was the larger part of the kernel's code and a good microsecond of every launch.
__device__ __forceinline__ int tile_chunk_begin(const TileParams& p, int i) {
    // balanced: floor(i units / nchunks) = i q + floor(i r / nchunks), units = q nchunks + r  (i r < nchunks^2)
    if (p.split_k == 0) return i * p.bal_q + fast_div(i * p.bal_r, p.div_nchunks);
    const int t = fast_div(i, p.div_split), s = i - t * p.split_k;
    return t * p.G + s * p.slice_base + min(s, p.slice_rem);
}
// The chunk that holds unit u.  (Out of line and with scalar arguments -- a reference to the kernel's parameter
// block would be copied to local memory for every call; only the Split-K epilogue of balanced chunks comes here.)
static __device__ __noinline__ int tile_chunk_of_s(int split_k, int G, int nchunks, long long units, long long u) {
    if (split_k == 0) return (int)(((u + 1) * nchunks - 1) / units);
    const int t = (int)(u / G), g = (int)(u - (long long)t * G);
    const int base = G / split_k, rem = G % split_k;
    const int s = (g < rem * (base + 1)) ? g / (base + 1) : rem + (g - rem * (base + 1)) / max(base, 1);
    return t * split_k + s;
}
__device__ __forceinline__ int tile_chunk_of(const TileParams& p, long long u) {
    return tile_chunk_of_s(p.split_k, p.G, p.nchunks, (long long)p.m_tiles * p.n_tiles * p.G, u);
}

// Where chunk ci (or the next non-empty one of this CTA, stepping by `stride`) starts.
struct ChunkStart {
    int ci;        // the chunk found (>= nchunks: none left)
    int t;         // tile = batch tile * NT + column tile
    int nt, mt_i;  // t % NT, t / NT
    int g0;        // first group inside the tile
    int len;       // units of the chunk
};
__device__ __forceinline__ ChunkStart tile_chunk_start(const TileParams& p, int ci, int stride) {
    ChunkStart c;
    int u0 = 0, len = 0;
    while (ci < p.nchunks) {
        u0 = tile_chunk_begin(p, ci);
        len = tile_chunk_begin(p, ci + 1) - u0;
        if (len > 0) break;
        ci += stride;
    }
    c.ci = ci;
    c.len = len;
    c.t = fast_div(u0, p.div_G);
    c.g0 = u0 - c.t * p.G;
    c.mt_i = fast_div(c.t, p.div_ntiles);
    c.nt = c.t - c.mt_i * p.n_tiles;
    return c;
}

// Walks the segments of this CTA's chunks in order (a segment = the part of a chunk inside one
// tile).  Every role of the CTA runs its own copy and sees the same sequence.  A warp runs dependent
// scalar code at only one instruction every several clocks, and the producer and MMA warps sit on
// the critical path of every stage: so all per-stage work of the roles is a plain counted loop over
// the segment's 2 * units stages, and the chunk arithmetic happens here, once per chunk.
struct SegWalk {
    const TileParams& p;
    int ci;            // current chunk
    int t;             // tile = batch tile * NT + column tile
    int nt, mt_i;      // t % NT, t / NT
    int g0;            // first group of the segment inside the tile
    int units;         // groups in the segment
    int left;          // units of the chunk after this segment
    bool first;        // first segment of its chunk
    uint32_t n0;       // stages of this CTA before the segment (ring positions derive from it)
    const int spu;     // stages per unit (group): 1 or 2
    __device__ __forceinline__ SegWalk(const TileParams& p_, int spu_)
        : p(p_), ci((int)blockIdx.x), t(0), nt(0), mt_i(0), g0(0), units(0), left(0), first(true), n0(0), spu(spu_) {
        load_chunk();
    }
    __device__ __forceinline__ void load_chunk() {
        const ChunkStart c = tile_chunk_start(p, ci, (int)gridDim.x);
        ci = c.ci;
        if (ci >= p.nchunks) return;
        t = c.t;
        g0 = c.g0;
        mt_i = c.mt_i;
        nt = c.nt;
        units = min(c.len, p.G - g0);
        left = c.len - units;
        first = true;
    }
    __device__ __forceinline__ bool valid() const { return ci < p.nchunks; }
    __device__ __forceinline__ void next() {
        n0 += (uint32_t)(spu * units);
        if (left == 0) {
            ci += (int)gridDim.x;
            load_chunk();
            return;
        }
        ++t;
        if (++nt == p.n_tiles) { nt = 0; ++mt_i; }
        g0 = 0;
        units = min(left, p.G);
        left -= units;
        first = false;
    }
    __device__ __forceinline__ int stages_in_seg() const { return spu * units; }
    __device__ __forceinline__ bool whole_tile() const { return g0 == 0 && units == p.G; }
};

// Position in the ring of R slots: slot = n % R, turn = n / R, phase = turn & 1, kept incrementally.
struct RingPos {
    int slot;
    uint32_t ph;
    uint32_t turn;
    __device__ __forceinline__ void advance(int d, int R) {
        slot += d;
        while (slot >= R) { slot -= R; ph ^= 1u; ++turn; }
    }
};

// "The MMAs that read this slot have retired" has TWO barriers per slot, used by alternate ring turns.
// A parity wait tells a phase from the one before it, not from the one two back, so whoever waits on
// a barrier must see every one of its phases.  The producer does (it walks every stage).  A dequant
// set takes every fourth stage, and with six slots it comes back to a slot only every second turn;
// with one barrier per slot it would skip a phase each time, and nothing but a single in-order issuer
// would keep the skipped phase from still being open.  With one barrier per slot and turn parity the
// set meets the same barrier on every visit and that barrier completes exactly one phase in between.
__device__ __forceinline__ uint64_t* retired_bar(uint64_t* retired, const RingPos& r) {
    return retired + (r.turn & 1u) * kTileMaxStages + r.slot;      // the stage at r commits here
}
// until the stage that used r's slot one ring turn earlier has retired (r.turn >= 1)
__device__ __forceinline__ bool wait_slot_free(uint64_t* retired, const RingPos& r) {
    const uint32_t t = r.turn - 1u;
    return mbar_wait(retired + (t & 1u) * kTileMaxStages + r.slot, (t >> 1) & 1u);
}

// Packed words, scales and zero points of one thread's column for one stage of 32 * NW k (NR
// quantization groups).
template <int NW, int NR>
struct StageRegs {
    uint4 w[NW];        // w[i]: k = 32 i .. 32 i + 31 of the stage
    uint32_t s[NR];     // 16-bit scale patterns
    uint32_t zw[NR];    // zero-point words that hold the column's nibble
};

// MT = batch rows per tile; SG = scale / zero-point rows per 128-k block (quantization group 128 / SG);
// BF = BF16 instead of FP16 activations, scales, weights and output; SYM = symmetric format (zero point 8,
// no Z buffer); EPI = bias / activation fused into the final cast.  (Both compiled in: decided at run time
// they cost 5 to 10 % on narrow tiles and 9 % at M = 256.)
template <int MT, int SG, bool BF, bool SYM, bool EPI>
__global__ void __launch_bounds__(tile_threads(MT), 1)
gemm_tile_kernel(const __grid_constant__ CUtensorMap tmap_a, const TileParams p) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    // 1024-byte alignment of the stage buffers (the swizzle atom) regardless of where the
    // dynamic segment starts
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    constexpr int kStageBytes = tile_stage_bytes(MT);
    constexpr uint32_t kIdesc = tile_idesc(MT, BF);
    constexpr int kCW = MT / kTileSets;                  // accumulator columns (batch rows) per epilogue warp
    constexpr int kNI = tile_issuers(MT);                // MMA-issuing warps, one accumulator (set) each
    constexpr int kDBufs = tile_dbufs(MT);               // accumulators per issuer: accumulator (b, i) sits
    constexpr int kDStride = tile_d_stride(MT);          // at column (b * kNI + i) * kDStride
    constexpr int kStageK = tile_stage_k(MT);            // k per ring slot
    constexpr int kSPU = kGroup / kStageK;               // stages per unit
    constexpr int kSlotCols = kStageK / 2;               // TMEM columns of one operand slot
    constexpr int kACol = tile_a_col_base(MT);
    constexpr int kNW = kStageK / 32;                    // 16-byte chunks of a thread's column per stage
    constexpr int kPF = tile_prefetch(MT);
    constexpr int kNR = SG / kSPU > 0 ? SG / kSPU : 1;   // scale rows one stage touches
    constexpr bool sym = SYM;

    uint64_t* full = reinterpret_cast<uint64_t*>(smem);          // [R]  activation box landed AND operand stored in TMEM
    uint64_t* retired = full + kTileMaxStages;                   // [2][R]  the stage's MMAs retired: slot free
    uint64_t* d_full = retired + 2 * kTileMaxStages;             // [2]  accumulator complete
    uint64_t* d_empty = d_full + 2;                              // [2]  accumulator drained by the epilogue
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(d_empty + 2);
    int* flags = reinterpret_cast<int*>(tmem_slot + 1);          // [0] a bounded wait ran out, [1] stages issued
    unsigned char* stage0 = smem + kTileBarBytes;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int R = p.stages;

    if (threadIdx.x == 0) {
        for (int i = 0; i < R; ++i) {
            mbar_init(&full[i], 1 + 4);      // the producer's arrive.expect_tx + one arrival per warp of a dequant set
            mbar_init(&retired[i], 1);
            mbar_init(&retired[kTileMaxStages + i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&d_full[i], kNI);      // every issuer reports once per segment
            mbar_init(&d_empty[i], kTileDequantWarps);
        }
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
    // the next kernel in the stream may start its own prologue and weight prefetch
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    if (warp == 0) {
        // ------------------------------------------------------------ producer: activation boxes
        if (elect_one()) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_a) : "memory");
        asm volatile("griddepcontrol.wait;" ::: "memory");   // activations may come from the previous kernel
        bool ok = true;
        RingPos r{0, 0u, 0u};
        uint32_t n = 0;
        for (SegWalk w(p, kSPU); w.valid() && ok; w.next()) {
            int kb = w.g0 * (kGroup / kTileBoxK);            // 64-k box index along K
            const int m = w.mt_i * MT;
            const int nst = w.stages_in_seg();
            for (int j = 0; j < nst; ++j) {
                if (r.turn != 0u && !wait_slot_free(retired, r)) { ok = false; break; }
                if (elect_one()) {
                    // one copy per stage: kStageK / 64 boxes of MT rows x 64 k, box b at b * MT * 128 bytes
                    mbar_expect_tx(&full[r.slot], (uint32_t)kStageBytes);
                    if constexpr (kStageK == kTileBoxK)
                        tma_load_2d(stage0 + (size_t)r.slot * kStageBytes, &tmap_a, kb * kTileBoxK, m, &full[r.slot]);
                    else
                        tma_load_3d(stage0 + (size_t)r.slot * kStageBytes, &tmap_a, 0, m, kb, &full[r.slot]);
                }
                __syncwarp();
                kb += kStageK / kTileBoxK;
                ++n;
                r.advance(1, R);
            }
        }
        if (lane == 0) {
            flags[1] = (int)n;
            if (!ok) *abort_flag = 1;
        }
    } else if (warp <= kNI) {
        // ------------------------------------------------------------ MMA issuer `iss`: the stages whose
        // index in this CTA is = iss (mod kNI), summed into this issuer's own accumulator
        const int iss = warp - 1;
        asm volatile("griddepcontrol.wait;" ::: "memory");
        uint32_t n_seg = 0, n_prev = 0;
        bool ok = true;
        RingPos r{0, 0u, 0u};
        for (SegWalk w(p, kSPU); w.valid() && ok; w.next(), ++n_seg) {
            const int dbuf = n_seg % kDBufs;
            // the epilogue of the segment that used this accumulator before must have drained it (an
            // issuer without a stage in this segment waits too, so that its report below cannot land
            // in the barrier phase of that earlier segment)
            if (!mbar_wait(&d_empty[dbuf], ((n_seg / kDBufs) & 1u) ^ 1u)) { ok = false; break; }
            const uint32_t d_t = tmem_base + (dbuf * kNI + iss) * kDStride;
            const int nst = w.stages_in_seg();
            int j = kNI == 1 ? 0 : (int)(((uint32_t)(iss + kNI) - w.n0 % kNI) % kNI);
            if (j >= nst) {
                if (elect_one()) mbar_arrive(&d_full[dbuf]);     // nothing of mine in this segment
                __syncwarp();
                continue;
            }
            uint32_t acc = 0u;                                   // the segment's first MMA overwrites
            for (; j < nst; j += kNI) {
                const uint32_t n = w.n0 + (uint32_t)j;
                r.advance((int)(n - n_prev), R);
                n_prev = n;
                if (!mbar_wait(&full[r.slot], r.ph)) { ok = false; break; }
                tc_fence_after();
                if (elect_one()) {
                    const uint64_t bdesc = smem_desc_sw128(smem_u32(stage0 + (size_t)r.slot * kStageBytes));
                    const uint32_t a_t = tmem_base + kACol + r.slot * kSlotCols;
#pragma unroll
                    for (int kk = 0; kk < kStageK / 16; ++kk) {
                        // 16 k per instruction: 8 TMEM columns of A; in B 32 bytes along the swizzled rows of
                        // a 64-k box, the next box MT * 128 bytes further
                        const uint64_t bd = bdesc + (uint64_t)((kk / 4) * (MT * 128 / 16) + (kk % 4) * 2);
                        tc_mma_ts(d_t, a_t + kk * 8, bd, kIdesc, kk == 0 ? acc : 1u);
                    }
                    tc_commit(retired_bar(retired, r));
                    if (j + kNI >= nst) tc_commit(&d_full[dbuf]);
                }
                __syncwarp();
                acc = 1u;
            }
        }
        if (!ok && lane == 0) *abort_flag = 1;
    } else {
        // ------------------------------------------------------------ dequant + epilogue warps
        const int dw = warp - (1 + kNI);       // 0..15
        const int set = dw >> 2;               // takes the stages whose index in this CTA is = set (mod 4)
        const int quarter = warp & 3;          // TMEM lanes this warp may touch
        const int row = quarter * 32 + lane;   // column n inside the CTA tile = TMEM lane
        const int half = row >> 6, col = row & 63;
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        // word offsets of this thread's two 16-byte chunks inside a block's 64-k half
        const int wo0 = (col >> 3) * 64 + (col & 7) * 4;
        const int wo1 = (col >> 3) * 64 + 32 + (((col & 7) + 4) & 7) * 4;
        const int zp = sz_perm(col);         // position of this column's scale / zero point inside a row
        const int zsh = 4 * (zp & 7);

        // this set's first stage inside a segment
        auto first_own = [&](const SegWalk& w) { return (int)(((uint32_t)set - w.n0) & 3u); };
        // Load cursor: runs kPF of this set's stages ahead of the compute loop.  Inside a segment this
        // set's stages are kTileSets apart (kTileSets / kSPU groups on, same part of the group), so the
        // three pointers just step; they are recomputed only when the cursor enters a new segment.
        SegWalk wl(p, kSPU);
        int jl = 0;
        bool l_in = false;                      // this thread's column exists (not past the matrix edge)
        const uint32_t* lw = nullptr;           // the stage's first word of this thread's 8-column block
        const uint16_t* ls = nullptr;
        const uint32_t* lz = nullptr;
        auto point = [&]() {                    // cursor entered a new segment: settle on a stage, set pointers
            while (wl.valid()) {
                jl = first_own(wl);
                if (jl < wl.stages_in_seg()) break;
                wl.next();
            }
            if (!wl.valid()) return;
            const int t64 = 2 * wl.nt + half;   // 64-column packed tile
            l_in = t64 * kTileN < p.N;
            const size_t blk = (size_t)t64 * p.G + (wl.g0 + jl / kSPU);
            lw = p.Wq + blk * kBlockWords + (jl % kSPU) * 512;
            // first scale row of the stage: a 64-k stage of a block with SG >= 2 rows starts at row (SG / 2) * half
            const size_t row = blk * SG + (SG >= kSPU ? (jl % kSPU) * (SG / kSPU) : 0);
            ls = p.S + row * kSBlockHalves + zp;
            lz = sym ? nullptr : p.Z + row * kZBlockWords + (zp >> 3);
        };
        // load the cursor's stage (zeros past the matrix edge) and advance the cursor
        auto fetch = [&](StageRegs<kNW, kNR>& r) {
            if (!wl.valid()) return;
            if (l_in) {
#pragma unroll
                for (int h = 0; h < kNW / 2; ++h) {
                    r.w[2 * h] = __ldg(reinterpret_cast<const uint4*>(lw + h * 512 + wo0));
                    r.w[2 * h + 1] = __ldg(reinterpret_cast<const uint4*>(lw + h * 512 + wo1));
                }
#pragma unroll
                for (int i = 0; i < kNR; ++i) {
                    r.s[i] = __ldg(ls + i * kSBlockHalves);
                    r.zw[i] = sym ? 0u : __ldg(lz + i * kZBlockWords);
                }
            } else {
#pragma unroll
                for (int i = 0; i < kNW; ++i) r.w[i] = make_uint4(0, 0, 0, 0);
#pragma unroll
                for (int i = 0; i < kNR; ++i) { r.s[i] = 0; r.zw[i] = 0; }
            }
            jl += kTileSets;
            if (jl < wl.stages_in_seg()) {
                lw += (kTileSets / kSPU) * kBlockWords;
                ls += (kTileSets / kSPU) * (SG * kSBlockHalves);
                if (!sym) lz += (kTileSets / kSPU) * (SG * kZBlockWords);
            } else {
                wl.next();
                point();
            }
        };
        point();
        // register ring of prefetched stages, written out so that no slot is ever copied
        static_assert(kPF == 2 || kPF == 3, "the ring below has two or three slots");
        StageRegs<kNW, kNR> pf0, pf1, pf2;
        fetch(pf0);
        fetch(pf1);
        if (kPF == 3) fetch(pf2);
        // Converting weights into the TMEM ring touches nothing the previous kernel may still be writing,
        // so it starts at once and runs until the ring is full; the dependency wait comes before this
        // warp's first write to global memory (the first epilogue).
        bool dep_waited = false;

        uint32_t n_seg = 0, n_prev = 0;
        int pi = 0;                             // ring slot that holds the next stage to convert
        RingPos rp{0, 0u, 0u};
        bool ok = true;
        // one stage of this thread's column -> kSlotCols TMEM columns of the ring slot
        auto convert = [&](const StageRegs<kNW, kNR>& cur, uint32_t n) -> bool {
            uint32_t s2[kNR], zlo[kNR], zhi[kNR];
#pragma unroll
            for (int i = 0; i < kNR; ++i) {
                const uint32_t z = sym ? (uint32_t)kSymZero : ((cur.zw[i] >> zsh) & 15u);
                s2[i] = cur.s[i] * 0x00010001u;
                zlo[i] = zconst_lo<BF>(z);
                zhi[i] = zconst_hi<BF>(z);
            }
            // the MMAs that read this slot one ring turn ago must have retired
            if (rp.turn != 0u && !wait_slot_free(retired, rp)) return false;
            tc_fence_after();
            const uint32_t a_t = tmem_base + lane_addr + kACol + rp.slot * kSlotCols;
#pragma unroll
            for (int c = 0; c < kNW; ++c) {      // 32 k -> 16 TMEM columns at a time
                const uint32_t ww[4] = {cur.w[c].x, cur.w[c].y, cur.w[c].z, cur.w[c].w};
                constexpr int kRowDiv = 4 / SG > 0 ? 4 / SG : 1;   // 32-k chunks per scale row (group / 32)
                const int ri = (c / kRowDiv) < kNR ? (c / kRowDiv) : kNR - 1;
                uint32_t regs[16];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const Pack8 f = dequant_word<BF>(ww[i], zlo[ri], zhi[ri], s2[ri]);
#pragma unroll
                    for (int q = 0; q < 4; ++q) regs[4 * i + q] = f.h[q];
                }
                tc_st16(a_t + 16 * c, regs);
            }
            return true;
        };
        for (SegWalk w(p, kSPU); w.valid() && ok; w.next(), ++n_seg) {
            const int nst = w.stages_in_seg();
            for (int j = first_own(w); j < nst; j += kTileSets) {
                const uint32_t n = w.n0 + (uint32_t)j;
                rp.advance((int)(n - n_prev), R);
                n_prev = n;
                // convert ring slot pi, then refill it with the stage kPF ahead
                if (pi == 0) { ok = convert(pf0, n); fetch(pf0); pi = 1; }
                else if (kPF == 2 || pi == 1) { ok = convert(pf1, n); fetch(pf1); pi = (kPF == 3) ? 2 : 0; }
                else {
                    if constexpr (kPF == 3) { ok = convert(pf2, n); fetch(pf2); }
                    pi = 0;
                }
                if (!ok) break;
                tc_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&full[rp.slot]);
            }
            if (!ok) break;

            // ---------------------------------------------------- epilogue of this segment
            const int dbuf = n_seg % kDBufs;
            if (!mbar_wait(&d_full[dbuf], (n_seg / kDBufs) & 1u)) { ok = false; break; }
            tc_fence_after();
            if (!dep_waited) {
                asm volatile("griddepcontrol.wait;" ::: "memory");
                dep_waited = true;
            }
            const int T = w.t;
            const int n = w.nt * kTileCols + row;
            const int m_base = w.mt_i * MT + set * kCW;     // first batch row of this warp's columns
            const uint32_t d_t = tmem_base + lane_addr + (dbuf * kNI) * kDStride + set * kCW;
            // first stage of each issuer inside this segment: an issuer with none has no sum to add
            const int iss0 = (int)(w.n0 % kNI);
            const long long tile_u0 = (long long)T * p.G;
            const bool whole = w.whole_tile();
            // first segment of a chunk -> slot 2 ci, its continuation into a later tile -> 2 ci + 1
            float* part = p.ws + ((size_t)(2 * w.ci + (w.first ? 0 : 1)) * MT + set * kCW) * kTileCols + row;
            constexpr int kStep = kCW >= 16 ? 16 : kCW;
#pragma unroll 1
            for (int cc = 0; cc < kCW; cc += kStep) {
                uint32_t v[kStep];
                if constexpr (kNI == 1) {
                    if constexpr (kStep == 16) tc_ld16(d_t + cc, v);
                    else if constexpr (kStep == 8) tc_ld8(d_t + cc, v);
                    else tc_ld4(d_t + cc, v);
                    tc_wait_ld();
                }
                // several issuers: add their sums in stage order (issuer iss0 took the segment's first stage)
#pragma unroll
                for (int ii = 0; ii < (kNI == 1 ? 0 : kNI); ++ii) {
                    if (ii >= nst) break;                        // warp-uniform
                    int i = iss0 + ii;
                    if (i >= kNI) i -= kNI;
                    uint32_t t[kStep];
                    if constexpr (kStep == 16) tc_ld16(d_t + i * kDStride + cc, t);
                    else if constexpr (kStep == 8) tc_ld8(d_t + i * kDStride + cc, t);
                    else tc_ld4(d_t + i * kDStride + cc, t);
                    tc_wait_ld();
#pragma unroll
                    for (int q = 0; q < kStep; ++q)
                        v[q] = ii == 0 ? t[q] : __float_as_uint(__uint_as_float(v[q]) + __uint_as_float(t[q]));
                }
                if (whole) {
                    if (n < p.N) {
#pragma unroll
                        for (int q = 0; q < kStep; ++q) {
                            const int m = m_base + cc + q;
                            if (m < p.M) p.C[(size_t)m * p.N + n] = (EPI ? finish<BF>(__uint_as_float(v[q]), n, p.epi) : cast_out<BF>(__uint_as_float(v[q])));
                        }
                    }
                } else {
#pragma unroll
                    for (int q = 0; q < kStep; ++q) part[(size_t)(cc + q) * kTileCols] = __uint_as_float(v[q]);
                }
            }
            // accumulator drained: a later segment's first MMA may overwrite it
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&d_empty[dbuf]);

            if (!whole && p.defer_reduce == 0) {
                // Split-K reduce (Algorithm 1, Phase 3), per warp region (32 columns n x MT/4 rows m)
                __threadfence();
                __syncwarp();
                // (classic slices: no division on the way to the ticket)
                const int c_first = p.split_k > 0 ? T * p.split_k : tile_chunk_of(p, tile_u0);
                const int c_last = p.split_k > 0 ? c_first + p.split_k - 1 : tile_chunk_of(p, tile_u0 + p.G - 1);
                int* ticket = p.tickets + ((size_t)T * kTileDequantWarps + dw);
                int last = 0;
                if (lane == 0) {
                    const int old = atomicAdd(ticket, 1);
                    last = (old == c_last - c_first);
                    if (last) *ticket = 0;   // every contributor has arrived: zero for the next call
                }
                last = __shfl_sync(0xffffffffu, last, 0);
                if (last) {
                    __threadfence();
                    // contributors in ascending K: chunk c_first (its first segment if it starts at the tile's
                    // first unit, else its continuation), then the first segments of the others.  Rows are
                    // summed kStep at a time so that many loads are in flight.
                    const size_t slot_elems = (size_t)MT * kTileCols;
                    const float* base = p.ws + (size_t)(set * kCW) * kTileCols + row;
                    const size_t first_slot =
                        2 * (size_t)c_first + ((p.split_k > 0 || tile_chunk_begin(p, c_first) == tile_u0) ? 0 : 1);
#pragma unroll 1
                    for (int m0 = 0; m0 < kCW; m0 += kStep) {
                        float acc[kStep];
#pragma unroll
                        for (int q = 0; q < kStep; ++q)
                            acc[q] = __ldcg(base + first_slot * slot_elems + (size_t)(m0 + q) * kTileCols);
                        // two contributors' loads in flight at a time (one per round trip would make
                        // the tail S - 1 trips long); the additions keep the ascending order
                        int c = c_first + 1;
                        for (; c + 1 <= c_last; c += 2) {
                            const float* src = base + (size_t)(2 * c) * slot_elems + (size_t)m0 * kTileCols;
                            float x0[kStep], x1[kStep];
#pragma unroll
                            for (int q = 0; q < kStep; ++q) {
                                x0[q] = __ldcg(src + (size_t)q * kTileCols);
                                x1[q] = __ldcg(src + 2 * slot_elems + (size_t)q * kTileCols);
                            }
#pragma unroll
                            for (int q = 0; q < kStep; ++q) { acc[q] += x0[q]; acc[q] += x1[q]; }
                        }
                        if (c <= c_last) {
                            const float* src = base + (size_t)(2 * c) * slot_elems + (size_t)m0 * kTileCols;
#pragma unroll
                            for (int q = 0; q < kStep; ++q) acc[q] += __ldcg(src + (size_t)q * kTileCols);
                        }
                        if (n < p.N) {
#pragma unroll
                            for (int q = 0; q < kStep; ++q) {
                                const int m = m_base + m0 + q;
                                if (m < p.M) p.C[(size_t)m * p.N + n] = (EPI ? finish<BF>(acc[q], n, p.epi) : cast_out<BF>(acc[q]));
                            }
                        }
                    }
                }
            }
        }
        if (!ok && lane == 0) *abort_flag = 1;
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (*abort_flag != 0 && threadIdx.x == 0) {
        // some wait ran out: before the CTA's shared memory goes away, give the copies still in
        // flight a (bounded) chance to land -- the last use of every ring slot.  (The phase may lack
        // the dequant warps' arrivals and then runs into the limit; the wait is bounded either way.)
        const uint32_t issued = (uint32_t)flags[1];
        for (uint32_t back = 0; back < (uint32_t)R && back < issued; ++back) {
            const uint32_t ns = issued - 1 - back;
            mbar_wait(&full[ns % R], (ns / R) & 1u);
        }
    }
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
    }
}

}  // namespace w4a16
