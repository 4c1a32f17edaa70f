// C ABI of the library (declared in include/w4a16.h): argument validation, per-shape
// kernel and Split-K selection, launches.  Every step of the computation runs in the
// kernels included below; this file only marshals arguments.
#include "w4a16.h"

#include <cuda_runtime.h>

#include <string.h>

#include <mutex>

#include "common.cuh"
#include "kernels_basic.cuh"
#include "kernel_tables.h"

using namespace w4a16;

namespace {

constexpr int kMaxDevices = 64;
constexpr size_t kWsHeaderBytes = 16384;  // zeroed ticket counters ahead of the FP32 partials
constexpr long kMaxTickets = kWsHeaderBytes / sizeof(int);

struct DeviceState {
    bool probed = false;
    bool is_sm100 = false;
    int sm_count = 148;
    int max_smem_optin = 0;
    void* ws = nullptr;
    size_t ws_bytes = 0;
    bool decode_attr_set[3][2][3][2][2][2] = {};   // [mb][cluster exchange][log2 SG][bf16][symmetric][tensor-copy rows]
    bool tile_attr_set[5][3][2][2][2] = {};   // [batch-tile index][log2 SG][bf16][symmetric][epilogue]
    // Programmatic dependent launch lets a GEMM kernel prefetch packed weights before the previous
    // kernel in its stream has finished.  The previous kernel of a stream may be a w4a16_pack that
    // writes those weights, so the first GEMM launched on a stream after any pack on the device is a
    // plain, fully ordered launch, and only the launches after it on that stream overlap their
    // predecessor again.  pack_epoch counts the packs; the table remembers, per stream, the epoch of
    // its last GEMM launch (a stream that is not in the table gets a plain launch).
    unsigned long long pack_epoch = 1;
    struct StreamEpoch { cudaStream_t stream; unsigned long long epoch; };
    static constexpr int kStreamSlots = 32;
    StreamEpoch streams[kStreamSlots] = {};
    int stream_evict = 0;
    bool cluster_ok = true;   // cleared when a cluster launch is refused (fewer SMs than usual, MPS limits ...)

    // May this launch on `st` overlap the previous kernel of the stream?  Records the launch.
    bool pdl_allowed(cudaStream_t st) {
        for (int i = 0; i < kStreamSlots; ++i) {
            if (streams[i].epoch != 0 && streams[i].stream == st) {
                const bool ok = streams[i].epoch == pack_epoch;
                streams[i].epoch = pack_epoch;
                return ok;
            }
        }
        int slot = -1;
        for (int i = 0; i < kStreamSlots; ++i)
            if (streams[i].epoch == 0) { slot = i; break; }
        if (slot < 0) { slot = stream_evict; stream_evict = (stream_evict + 1) % kStreamSlots; }
        streams[slot].stream = st;
        streams[slot].epoch = pack_epoch;
        return false;
    }
};
DeviceState g_dev[kMaxDevices];
// One lock for the per-device records above (workspace registration, attribute flags, stream table):
// the entry points may be called from several host threads.
std::mutex g_mu;

int current_device(DeviceState** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        cudaGetLastError();
        return W4A16_ERR_CUDA;
    }
    DeviceState& d = g_dev[dev];
    if (!d.probed) {
        int major = 0, sms = 0, smem = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) {
            cudaGetLastError();
            return W4A16_ERR_CUDA;
        }
        d.is_sm100 = (major == 10);
        d.sm_count = sms > 0 ? sms : 148;
        d.max_smem_optin = smem;
        d.probed = true;
    }
    *out = &d;
    return W4A16_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_weight_shape(int N, int K, int group) {
    if (!group_ok(group)) return W4A16_ERR_SHAPE;
    if (K <= 0 || N <= 0 || K % kGroup != 0 || N % kTileN != 0) return W4A16_ERR_SHAPE;
    return W4A16_OK;
}
int log2_sg(int sg) { return sg == 1 ? 0 : sg == 2 ? 1 : 2; }
bool flags_ok(int flags) { return (flags & ~(W4A16_FLAG_SYMMETRIC | W4A16_FLAG_BF16)) == 0; }

size_t round256(size_t b) { return (b + 255) / 256 * 256; }

int sm_count_or_default() {
    DeviceState* d = nullptr;
    if (current_device(&d) == W4A16_OK) return d->sm_count;
    return 148;
}

// ---- decode-path launch geometry ------------------------------------------------
int decode_mb(int M) { return M <= 8 ? 1 : 2; }

// The decode kernel is persistent: `ctas` CTAs per batch chunk (two per SM with about 100 KiB of
// shared memory each, or three with about 60 KiB; 9 warps), `nchunks` chunks of work units dealt to
// them.
struct DecodeGeom {
    int mb, mchunks, stages, smem_bytes, ctas, nchunks;
    int stage_bytes;   // ring stride for the batch rows a CTA has
    int prefetch;      // stages whose weights are requested before the wait for the previous kernel
    bool a_box;        // activation rows of a stage as one tensor copy (kernel_decode.cuh)
    int cps;       // CTAs per SM the launch is sized for (2 or 3)
    bool cluster;  // one thread-block cluster of split_k CTAs per tile: partial tiles meet in shared memory
    int split_k;   // what the kernel runs: 0 = balanced chunks, S >= 1 = S slices per tile
};

// From how many batch rows per CTA on a stage's activation rows come as one tensor copy instead of one bulk
// copy per row.  Measured (us, bulk copies per row / one tensor copy), K = 11008 / N = 4096: M = 2 9.28 / 9.09,
// M = 4 9.60 / 9.09, M = 8 10.5 / 9.34, M = 16 13.0 / 11.1; K = 4096 / N = 4096, M = 3: 5.57 / 5.38.  With one
// row the two are within 1 % (9.15 / 9.09 there, 32.6 / 32.8 at K = 28672 / N = 8192, 14.9 / 15.2 at K = 4096 /
// N = 22016: the box takes 8 KiB of a slot whatever M is, and long shapes want the ring stage that costs).
constexpr int kDecABoxMinRows = 2;

DecodeGeom decode_geom(int M, int N, int G, int split_k, int sms, bool allow_cluster = true, int sg = 1) {
    DecodeGeom g;
    g.mb = decode_mb(M);
    g.mchunks = (M + 8 * g.mb - 1) / (8 * g.mb);
    const int T = N / kTileN;
    const long units = (long)T * G;
    // Two CTAs per SM.  (Three, with a two-stage ring and 72 registers, were ahead on long launches
    // while every exchange went through the workspace; with the cluster exchange two are ahead again
    // everywhere but K = 4096 / N = 12288, by 3 %: 33.8 against 34.8 us at K = 28672 / N = 8192, 15.0
    // against 15.8 at N = 22016.  The kernel keeps the template parameter.)
    g.cps = 2;
    long slots = (long)g.cps * sms;
    if (split_k == 0) {
        // How the unit range is cut when the caller leaves it open.  Balanced chunks use every CTA
        // slot, but a chunk that crosses a tile boundary goes through the workspace exchange in
        // mid-stream.  S slices per tile keep every chunk inside one tile, and their exchange is
        // cheaper: none at S = 1, through the cluster for S <= 6, at the end of the stream otherwise.
        // Slices are sized for 7/8 of the slots: a launch that fills every slot cannot start (and
        // prefetch its weights) before the launch in front of it has drained (K = 10240 / N = 4608,
        // 72 tiles: three slices 10.7 us, four 13.2).  Costs in units per CTA, exchanges priced from
        // measurements: none 0, cluster 4, workspace at the end of a slice 9, workspace in mid-stream
        // 13 (1.3 / 2.8 / about 4 us at 0.3 us per unit).  K = 4096 / N = 22016: whole tiles 15.0 us,
        // balanced 18.1; K = 28672 / N = 8192: two slices 33.8, balanced 34.3; K = 11008 / N = 4096:
        // four slices 9.7, three 10.5, two 13.5; K = 6144 / N = 1536: six slices in a cluster 4.8,
        // twelve through the workspace 6.5.  Equal chunks over every slot also run 8 % longer than their
        // share of the units says (SMs finish the same work up to 8 % apart, and with every slot taken there
        // is no slack): K = 28672 / N = 8192 balanced 32.4 / two slices in a cluster 31.7 us at M = 1, 40.6 /
        // 38.7 at M = 16; K = 22016 / N = 8192 26.6 / 25.1; but K = 8192 / N = 10240 balanced 16.5 / whole 18.7.
        long best = (units * 27 / 25 + slots - 1) / slots + 13;
        int best_s = 0;
        if (T > slots) {
            // more tiles than CTAs: whole tiles dealt round-robin; the CTAs of an SM share its issue
            // slots, so uneven tile counts cost less than the longest CTA suggests (15 % allowed)
            const long whole_cost = (units * 23 / 20 + slots - 1) / slots;
            if (whole_cost <= best) { best = whole_cost; best_s = 1; }
        } else {
            int s0 = (int)((slots * 7 / 8) / T);
            if (s0 < 1) s0 = 1;
            if (s0 > G) s0 = G;
            const long ws_cost = (G + s0 - 1) / s0 + (s0 == 1 ? 0 : 9);
            if (ws_cost <= best) { best = ws_cost; best_s = s0; }
            if (allow_cluster && g.mchunks == 1 && s0 >= 2) {
                const int sc = s0 < kDecMaxCluster ? s0 : kDecMaxCluster;   // fewer, longer slices that fit a cluster
                const long cl_cost = (G + sc - 1) / sc + 4;
                if (cl_cost <= best) { best = cl_cost; best_s = sc; }
            }
        }
        split_k = best_s;
    }
    g.split_k = split_k;
    if (split_k == 0) {
        // balanced chunks, one per CTA; no more CTAs than stages' worth of units
        long want = (units + kDecUnitsPerStage - 1) / kDecUnitsPerStage;
        g.ctas = (int)(want < slots ? want : slots);
        if (g.ctas < 1) g.ctas = 1;
        g.nchunks = g.ctas;
    } else {
        g.nchunks = T * split_k;
        g.ctas = (int)((long)g.nchunks < slots ? (long)g.nchunks : slots);
    }
    // S slices per tile, every slice on a CTA of its own, one batch chunk: the S CTAs of a tile form a
    // cluster and exchange their partial tiles through distributed shared memory
    g.cluster = allow_cluster && split_k >= 2 && split_k <= kDecMaxCluster && g.nchunks == g.ctas && g.mchunks == 1;
    const int budget = (227 * 1024) / g.cps - 1024;   // per CTA
    const int xs = g.cluster ? split_k : 0;   // slices that meet in the exchange buffer
    const int rows = M < 8 * g.mb ? M : 8 * g.mb;   // batch rows of a CTA (the last chunk of a large M may have fewer)
    // (the box is 8 chunks of 64 k long: K >= 512)
    g.a_box = rows >= kDecABoxMinRows && G >= kDecUnitsPerStage;
    g.stage_bytes = decode_stage_bytes(rows, sg, g.a_box);
    int st = kDecMaxStages;
    while (st > 2 && decode_smem_bytes(g.mb, rows, sg, st, xs, g.a_box) > budget) --st;
    g.stages = st;
    // Weights do not depend on the previous kernel of the stream, so they may be requested before the wait
    // for it.  With K slices that pays only for about as many bytes as HBM delivers during that wait (about
    // 1 us, 6.5 MB over the whole grid): requests beyond that take bandwidth from the previous kernel's last
    // CTAs and stand in the copy queue in front of this kernel's activation rows.  Measured, stages requested
    // early = 1 / 2 / whole ring: K = 11008 / N = 4096 (256 CTAs), M = 1: 9.15 / 9.4 / 10.4 us; K = 16384 /
    // N = 4096: 11.7 / 12.0 / 12.9; K = 6144 / N = 1536 (144 CTAs), M = 8: 5.7 / 5.25 / 5.25.  Whole tiles
    // (wide N, split_k = 1) gain 2 to 4 % from the whole ring (K = 4096 / N = 22016: 15.45 / 15.2 / 14.9 us).
    {
        const long stage_w = (long)kDecUnitsPerStage * (kBlockBytes + sg * (kSBlockHalves * 2 + kZBlockWords * 4));
        long pf = 6500000L / ((long)g.ctas * g.mchunks * stage_w);
        if (pf < 1) pf = 1;
        if (pf > st || split_k == 1) pf = st;
        g.prefetch = (int)pf;
    }
    g.smem_bytes = decode_smem_bytes(g.mb, rows, sg, g.stages, xs, g.a_box);
    return g;
}

// Nominal split factor of the balanced schedule: how many CTAs share one column tile's K range.
int choose_split_decode(int M, int N, int G, int sms) {
    DecodeGeom g = decode_geom(M, N, G, 0, sms);
    if (g.split_k >= 1) return g.split_k;
    const int T = N / kTileN;
    int s = (g.ctas + T - 1) / T;
    if (s < 1) s = 1;
    if (s > G) s = G;
    return s;
}

// ---- tile-path launch geometry ----------------------------------------------------
// MT (batch rows per CTA tile = UMMA N) is the smallest of 16, 32, 64, 128, 256 that covers M, else
// 256.  The unit range (batch tile x column tile x group) is cut into `nchunks` chunks for `ctas`
// persistent CTAs: balanced chunks, one per CTA, when the caller leaves split_k open; S slices
// per tile otherwise.
struct TileGeom {
    int mt, mt_index, m_tiles, n_tiles, split_k, nchunks, stages, smem_bytes, ctas;
    long tiles;
};

constexpr size_t kTileTicketBytes = 131072;   // 16 counters per tile, after the 16 KiB of the small-M kernel
constexpr size_t kWsFullHeaderBytes = kWsHeaderBytes + kTileTicketBytes;
constexpr long kTileMaxTicketTiles = kTileTicketBytes / (sizeof(int) * kTileDequantWarps);

// Batch rows per CTA tile: the smallest of 16 .. 256 that covers M -- except that a narrow weight
// matrix gives such tiles too few of them for 148 SMs (N = 1536 and M = 64: twelve), and where the Split-K
// sum is made inside the kernel a twelve-way split costs more than converting the weights once per narrower
// batch tile: M = 64, N = 1536: 14.5 us with 64-row tiles, 10.1 with 32; M = 32: 10.7 against 9.0 with 16.
// With 24 tiles or fewer, take the widest narrower tile that gives at least 24.  Tiles of 128 and 256 rows
// hand that sum to a second kernel, so from twelve column tiles on they stay (us with 64- / 128- / 256-row
// tiles: M = 256: K = 8192 / N = 2048 19.1 / 17.1 / 16.1, K = 10240 / N = 2048 21.9 / 19.4 / 17.0, K = 8192 /
// N = 3072 26.8 / 20.9 / 18.6; M = 512, K = 6144 / N = 1536 23.1 / 17.6 / 16.5; M = 128: K = 8192 / N = 2048
// 13.6 / 13.3 / 15.1, K = 6144 / N = 1536 12.2 / 11.8 / 13.3); with eight column tiles the narrow tile is still
// ahead (M = 256, K = 4096 / N = 1024: 10.6 / 11.0 / 12.6).
int tile_mt_index(int M, int N) {
    const int idx = M <= 16 ? 0 : M <= 32 ? 1 : M <= 64 ? 2 : M <= 128 ? 3 : 4;
    const long n_tiles = (N + kTileCols - 1) / kTileCols;
    auto tiles = [&](int i) { return (long)((M + (16 << i) - 1) / (16 << i)) * n_tiles; };
    if (tiles(idx) > 24) return idx;
    if (idx >= 3 && n_tiles >= 12) return idx;
    for (int i = idx - 1; i >= 0; --i) {
        if (i == 3) continue;   // (128 rows were slower than 64 wherever the narrower tile was taken)
        if (tiles(i) >= 24) return i;
    }
    return 0;   // even 16-row tiles are few: take the most there are
}

TileGeom tile_geom(int M, int N, int G, int split_k, int sms, int max_smem) {
    TileGeom g;
    g.mt_index = tile_mt_index(M, N);
    g.mt = 16 << g.mt_index;
    g.m_tiles = (M + g.mt - 1) / g.mt;
    g.n_tiles = (N + kTileCols - 1) / kTileCols;
    g.tiles = (long)g.m_tiles * g.n_tiles;
    // more tiles than ticket counters: whole tiles only (no partial tiles, no tickets)
    if (split_k == 0 && g.tiles > kTileMaxTicketTiles) split_k = 1;
    if (split_k == 0) {
        // Balanced chunks use every SM to the end, but a chunk that starts or ends inside a tile leaves
        // an FP32 partial tile behind (store, ticket, reload: the larger the batch tile the dearer, and
        // in mid-stream it stalls the pipeline).  S slices per tile (tiles <= SMs) or whole tiles in
        // waves (tiles > SMs) avoid that at the price of idle SMs.  Cost model in groups per CTA; the
        // constants are fitted to measurements (K = 11008 / N = 4096, K = 28672 / N = 8192 and
        // K = N = 8192 with M up to 4096).
        // (narrow tiles: K = 4096 / N = 12288, M = 16: 96 whole tiles 13.8 us, balanced chunks 16.3)
        const long penalty = (g.mt <= 32 ? 10 : 6) + g.mt / 8;
        const long balanced_cost = (g.tiles * G + sms - 1) / sms + penalty;
        int s0 = 1;
        long classic_cost;
        if (g.tiles <= sms) {
            s0 = sms / (int)g.tiles;
            if (s0 > G) s0 = G;
            classic_cost = (G + s0 - 1) / s0;
        } else {
            classic_cost = ((g.tiles + sms - 1) / sms) * G;
        }
        if (classic_cost <= balanced_cost) split_k = s0;
    }
    g.split_k = split_k;
    if (split_k == 0) {
        const long units = g.tiles * G;
        long n = units / 2;                      // at least two units (four stages) per chunk
        if (n < 1) n = 1;
        if (n > sms) n = sms;
        g.nchunks = (int)n;
    } else {
        g.nchunks = (int)(g.tiles * split_k);
    }
    g.ctas = g.nchunks < sms ? g.nchunks : sms;
    const int avail = max_smem - kTileBarBytes - 1024;   // barrier block + alignment slack
    int st = avail / tile_stage_bytes(g.mt);
    if (st > kTileMaxStages) st = kTileMaxStages;
    if (st > tile_max_slots(g.mt)) st = tile_max_slots(g.mt);   // the ring also lives in tensor memory
    // parity waits tell a barrier phase only from its neighbour: every issuer has to come back to a slot
    // on every ring turn and every dequant set on every turn or every second one (kernel_tile.cuh)
    const int ring_unit = tile_issuers(g.mt) % 2 == 0 ? tile_issuers(g.mt) : 2 * tile_issuers(g.mt);
    st -= st % ring_unit;                                        // 0 (no valid ring) is refused by the caller
    g.stages = st;
    g.smem_bytes = kTileBarBytes + 1024 + st * tile_stage_bytes(g.mt);
    // each CTA takes the SM's whole tensor memory: ask for enough shared memory that two never share an SM
    if (g.smem_bytes < 120 * 1024) g.smem_bytes = 120 * 1024;
    return g;
}

// Partial-tile slots of the tile path: two per chunk.  Nothing when every chunk is a whole tile.
size_t tile_workspace_bytes(const TileGeom& g) {
    if (g.split_k == 1) return 0;
    return round256((size_t)2 * g.nchunks * g.mt * kTileCols * sizeof(float));
}

// Nominal split factor of the tile path's schedule: how many chunks share one tile's K range.
int choose_split_tile(int M, int N, int G, int sms) {
    TileGeom g = tile_geom(M, N, G, 0, sms, 227 * 1024);
    if (g.split_k >= 1) return g.split_k;
    long s = (g.nchunks + g.tiles - 1) / g.tiles;
    if (s < 1) s = 1;
    if (s > G) s = G;
    return (int)s;
}

// cuTensorMapEncodeTiled, resolved through the runtime so that libcuda is not a link dependency.
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (fn == nullptr) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
        else
            cudaGetLastError();
    }
    return fn;
}

// Activations A [M, K] FP16 row-major as a 2-D tensor (k innermost), box = 64 k x mt rows, 128-byte
// swizzle; rows past M read as zero.
bool make_act_tensor_map(CUtensorMap* map, const void* A, int M, int K, int mt) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (fn == nullptr) return false;
    if (tile_stage_k(mt) == kTileBoxK) {     // one box per stage: plain 2-D tensor, k innermost
        const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)M};
        const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
        const cuuint32_t box[2] = {(cuuint32_t)kTileBoxK, (cuuint32_t)mt};
        const cuuint32_t estr[2] = {1, 1};
        return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(A), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    }
    // A[M][K] seen as [K / 64][M][64]: one copy brings a stage's 64-k boxes one after the other
    const cuuint64_t dims[3] = {(cuuint64_t)kTileBoxK, (cuuint64_t)M, (cuuint64_t)(K / kTileBoxK)};
    const cuuint64_t strides[2] = {(cuuint64_t)K * 2, (cuuint64_t)kTileBoxK * 2};
    const cuuint32_t box[3] = {(cuuint32_t)kTileBoxK, (cuuint32_t)mt, (cuuint32_t)(tile_stage_k(mt) / kTileBoxK)};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<void*>(A), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The same activations for the warp-MMA kernel's tensor copy: [K / 64][M][64], box = the 8 chunks of a
// stage x 8 mb rows x 64 k.
bool make_decode_tensor_map(CUtensorMap* map, const void* A, int M, int K, int mb) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (fn == nullptr) return false;
    const cuuint64_t dims[3] = {64, (cuuint64_t)M, (cuuint64_t)(K / 64)};
    const cuuint64_t strides[2] = {(cuuint64_t)K * 2, 128};
    const cuuint32_t box[3] = {64, (cuuint32_t)(8 * mb), (cuuint32_t)kDecABoxChunks};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<void*>(A), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Path taken when the caller does not force one.  Measured on B200 (us, warp-MMA kernel / tcgen05 kernel): up to
// 16 batch rows the warp-MMA kernel is ahead or level everywhere, with or without a cluster exchange (M = 16:
// K = 11008 / N = 4096 10.8 / 12.2, K = N = 4096 6.0 / 7.9, K = 4096 / N = 12288 12.5 / 13.1, K = 4096 /
// N = 22016 18.8 / 21.7, K = 28672 / N = 8192 40.6 / 41.2, K = 18432 / N = 7168 26.4 / 26.7); from 17 rows on it
// needs a second pass over the weights and the tcgen05 kernel wins by 1.4 to 2 times (M = 24: 22.5 / 12.8 and
// 75.8 / 42.2 on the first and the last of those shapes).
int resolve_path(int M, int path) {
    if (path != W4A16_PATH_AUTO) return path;
    return M <= 16 ? W4A16_PATH_DECODE : W4A16_PATH_TILE;
}

// FP32 partials of the two-kernel reduce used by the plain path: [split_k][M][N].
size_t simple_partial_bytes(int M, int N, int split_k) {
    return round256((size_t)split_k * (size_t)M * (size_t)N * sizeof(float));
}
// Partial-tile slots of the decode kernel: [m chunk][2 * nchunks][8 mb][64] FP32.
size_t decode_partial_bytes(const DecodeGeom& g) {
    return round256((size_t)g.mchunks * 2 * (size_t)g.nchunks * (8 * g.mb) * kTileN * sizeof(float));
}

// ---- built-in scratch for w4a16_gemm_static_ws -------------------------------------
// Lives in the library's device image: every GPU that loads the library holds these bytes until
// the process exits.  In host code `g_static_ws` is only a handle for cudaGetSymbolAddress; the
// device address is looked up once per device (below) and that is what the kernel receives.
static __device__ __align__(256) unsigned char g_static_ws[W4A16_STATIC_WS_BYTES];
unsigned char* g_static_ws_addr[kMaxDevices] = {};

}  // namespace

// =====================================================================================
extern "C" {

const char* w4a16_strerror(int code) {
    switch (code) {
        case W4A16_OK: return "ok";
        case W4A16_ERR_NULL: return "null pointer argument";
        case W4A16_ERR_SHAPE: return "unsupported shape or option (need group in {32, 64, 128}, K % 128 == 0, N % 64 == 0, M >= 1)";
        case W4A16_ERR_ALIGN: return "buffer not 16-byte aligned (workspace: 256-byte)";
        case W4A16_ERR_SPLITK: return "split_k out of range for this shape / path";
        case W4A16_ERR_WORKSPACE: return "split-K workspace missing or too small (w4a16_set_workspace)";
        case W4A16_ERR_CUDA: return "CUDA runtime call failed";
        case W4A16_ERR_ARCH: return "current device is not sm_100";
        case W4A16_ERR_DEVICE_STATUS: return "a kernel gave up on a bounded wait";
        case W4A16_ERR_PATH: return "requested kernel path does not support this shape";
        default: return "unknown error code";
    }
}

size_t w4a16_packed_wq_bytes(int N, int K, int group) {
    if (check_weight_shape(N, K, group) != W4A16_OK) return 0;
    return (size_t)K * (size_t)N / 2;
}
size_t w4a16_packed_s_bytes(int N, int K, int group) {
    if (check_weight_shape(N, K, group) != W4A16_OK) return 0;
    return (size_t)(K / group) * (size_t)N * 2;
}
size_t w4a16_packed_z_bytes(int N, int K, int group) {   // asymmetric formats; a symmetric one has no Z buffer
    if (check_weight_shape(N, K, group) != W4A16_OK) return 0;
    return (size_t)(K / group) * (size_t)N / 2;
}

int w4a16_choose_split_k_ex(int M, int N, int K, int group, int path) {
    std::lock_guard<std::mutex> lock(g_mu);
    if (check_weight_shape(N, K, group) != W4A16_OK || M < 1) return 1;
    int G = K / kGroup;
    switch (resolve_path(M, path)) {
        case W4A16_PATH_DECODE: return choose_split_decode(M, N, G, sm_count_or_default());
        case W4A16_PATH_TILE: return choose_split_tile(M, N, G, sm_count_or_default());
        default: return 1;
    }
}
int w4a16_choose_path(int M, int N, int K, int group) {
    std::lock_guard<std::mutex> lock(g_mu);
    if (check_weight_shape(N, K, group) != W4A16_OK || M < 1) return W4A16_ERR_SHAPE;
    return resolve_path(M, W4A16_PATH_AUTO);
}
int w4a16_choose_split_k(int M, int N, int K, int group) {
    return w4a16_choose_split_k_ex(M, N, K, group, W4A16_PATH_AUTO);
}

size_t w4a16_workspace_bytes(int M, int N, int K, int group, int split_k) {
    std::lock_guard<std::mutex> lock(g_mu);
    if (check_weight_shape(N, K, group) != W4A16_OK || M < 1 || split_k < 0 || split_k > K / kGroup) return 0;
    // enough for whichever path w4a16_gemm / w4a16_gemm_ex may take with this split_k
    size_t need = 0;
    if (split_k != 1) {
        // the schedule differs between a device that places clusters and one that refused them: cover both
        DecodeGeom g = decode_geom(M, N, K / kGroup, split_k, sm_count_or_default(), true);
        DecodeGeom g2 = decode_geom(M, N, K / kGroup, split_k, sm_count_or_default(), false);
        need = decode_partial_bytes(g);
        if (g2.split_k != 1 && decode_partial_bytes(g2) > need) need = decode_partial_bytes(g2);
        int s = split_k == 0 ? choose_split_decode(M, N, K / kGroup, sm_count_or_default()) : split_k;
        size_t simple = simple_partial_bytes(M, N, s);
        if (simple > need) need = simple;
        TileGeom tg = tile_geom(M, N, K / kGroup, split_k, sm_count_or_default(), 227 * 1024);
        if (tile_workspace_bytes(tg) > need) need = tile_workspace_bytes(tg);
    }
    return need == 0 ? 0 : kWsFullHeaderBytes + need;
}

int w4a16_set_workspace(void* dev_ptr, size_t bytes) {
    std::lock_guard<std::mutex> lock(g_mu);
    DeviceState* d = nullptr;
    int rc = current_device(&d);
    if (rc != W4A16_OK) return rc;
    if (dev_ptr == nullptr || bytes == 0) {
        d->ws = nullptr;
        d->ws_bytes = 0;
        return W4A16_OK;
    }
    if ((reinterpret_cast<uintptr_t>(dev_ptr) & 255u) != 0) return W4A16_ERR_ALIGN;
    if (bytes < kWsFullHeaderBytes) return W4A16_ERR_WORKSPACE;
    // both kernels' ticket blocks start at zero (and leave zeros behind after every call)
    if (cudaMemset(dev_ptr, 0, kWsFullHeaderBytes) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) {
        cudaGetLastError();
        return W4A16_ERR_CUDA;
    }
    d->ws = dev_ptr;
    d->ws_bytes = bytes;
    return W4A16_OK;
}

int w4a16_quantize(const uint16_t* W16, uint32_t* Wq_raw, uint16_t* S_raw, uint8_t* Z_raw, int N, int K, int group,
                   int flags, w4a16_stream_t stream) {
    std::lock_guard<std::mutex> lock(g_mu);
    if (!flags_ok(flags)) return W4A16_ERR_SHAPE;
    const bool sym = (flags & W4A16_FLAG_SYMMETRIC) != 0, bf = (flags & W4A16_FLAG_BF16) != 0;
    if (!W16 || !Wq_raw || !S_raw || (!sym && !Z_raw)) return W4A16_ERR_NULL;
    int rc = check_weight_shape(N, K, group);
    if (rc != W4A16_OK) return rc;
    if (!aligned16(W16) || !aligned16(Wq_raw) || !aligned16(S_raw) || (!sym && !aligned16(Z_raw))) return W4A16_ERR_ALIGN;
    DeviceState* d = nullptr;
    if ((rc = current_device(&d)) != W4A16_OK) return rc;
    if (!d->is_sm100) return W4A16_ERR_ARCH;
    const int G = K / group;
    const size_t total = (size_t)G * N;
    const unsigned blocks = (unsigned)((total + 127) / 128);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint8_t* z = sym ? nullptr : Z_raw;
    if (bf) quantize_kernel<true><<<blocks, 128, 0, st>>>(W16, Wq_raw, S_raw, z, N, G, group, sym ? 1 : 0);
    else quantize_kernel<false><<<blocks, 128, 0, st>>>(W16, Wq_raw, S_raw, z, N, G, group, sym ? 1 : 0);
    return cudaGetLastError() == cudaSuccess ? W4A16_OK : W4A16_ERR_CUDA;
}

int w4a16_pack_fmt(const uint32_t* Wq_raw, const uint16_t* S_raw, const uint8_t* Z_raw, void* Wq, void* S, void* Z,
                   int N, int K, int group, int flags, w4a16_stream_t stream) {
    std::lock_guard<std::mutex> lock(g_mu);
    if (!flags_ok(flags)) return W4A16_ERR_SHAPE;
    const bool sym = (flags & W4A16_FLAG_SYMMETRIC) != 0;
    if (!Wq_raw || !S_raw || !Wq || !S) return W4A16_ERR_NULL;
    if (!sym && (!Z_raw || !Z)) return W4A16_ERR_NULL;
    int rc = check_weight_shape(N, K, group);
    if (rc != W4A16_OK) return rc;
    if (!aligned16(Wq_raw) || !aligned16(S_raw) || !aligned16(Wq) || !aligned16(S)) return W4A16_ERR_ALIGN;
    if (!sym && (!aligned16(Z_raw) || !aligned16(Z))) return W4A16_ERR_ALIGN;
    DeviceState* d = nullptr;
    if ((rc = current_device(&d)) != W4A16_OK) return rc;
    if (!d->is_sm100) return W4A16_ERR_ARCH;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int G = K / kGroup, sg = kGroup / group;
    size_t words = (size_t)K * N / 8, sc = (size_t)G * sg * N, zw = sc / 8;
    pack_wq_kernel<<<(unsigned)((words + 255) / 256), 256, 0, st>>>(Wq_raw, static_cast<uint32_t*>(Wq), N, G, words);
    pack_s_kernel<<<(unsigned)((sc + 255) / 256), 256, 0, st>>>(S_raw, static_cast<uint16_t*>(S), N, G, sg, sc);
    if (!sym)
        pack_z_kernel<<<(unsigned)((zw + 255) / 256), 256, 0, st>>>(Z_raw, static_cast<uint32_t*>(Z), N, G, sg, zw);
    ++d->pack_epoch;
    return cudaGetLastError() == cudaSuccess ? W4A16_OK : W4A16_ERR_CUDA;
}

int w4a16_pack(const uint32_t* Wq_raw, const uint16_t* S_raw, const uint8_t* Z_raw, void* Wq, void* S, void* Z,
               int N, int K, int group, w4a16_stream_t stream) {
    if (!Z_raw || !Z) return W4A16_ERR_NULL;
    return w4a16_pack_fmt(Wq_raw, S_raw, Z_raw, Wq, S, Z, N, K, group, 0, stream);
}

int w4a16_dequant_fmt(const void* Wq, const void* S, const void* Z, uint16_t* W16, int N, int K, int group, int flags,
                      w4a16_stream_t stream) {
    std::lock_guard<std::mutex> lock(g_mu);
    if (!flags_ok(flags)) return W4A16_ERR_SHAPE;
    const bool sym = (flags & W4A16_FLAG_SYMMETRIC) != 0, bf = (flags & W4A16_FLAG_BF16) != 0;
    if (!Wq || !S || !W16 || (!sym && !Z)) return W4A16_ERR_NULL;
    int rc = check_weight_shape(N, K, group);
    if (rc != W4A16_OK) return rc;
    if (!aligned16(Wq) || !aligned16(S) || (!sym && !aligned16(Z)) || !aligned16(W16)) return W4A16_ERR_ALIGN;
    DeviceState* d = nullptr;
    if ((rc = current_device(&d)) != W4A16_OK) return rc;
    if (!d->is_sm100) return W4A16_ERR_ARCH;
    size_t words = (size_t)K * N / 8;
    const uint32_t* z = sym ? nullptr : static_cast<const uint32_t*>(Z);
    const unsigned blocks = (unsigned)((words + 255) / 256);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (bf)
        dequant_kernel<true><<<blocks, 256, 0, st>>>(static_cast<const uint32_t*>(Wq), static_cast<const uint16_t*>(S), z,
                                                     W16, N, K / kGroup, kGroup / group, words);
    else
        dequant_kernel<false><<<blocks, 256, 0, st>>>(static_cast<const uint32_t*>(Wq), static_cast<const uint16_t*>(S), z,
                                                      W16, N, K / kGroup, kGroup / group, words);
    return cudaGetLastError() == cudaSuccess ? W4A16_OK : W4A16_ERR_CUDA;
}

int w4a16_dequant(const void* Wq, const void* S, const void* Z, uint16_t* W16, int N, int K, int group,
                  w4a16_stream_t stream) {
    if (!Z) return W4A16_ERR_NULL;
    return w4a16_dequant_fmt(Wq, S, Z, W16, N, K, group, 0, stream);
}

}  // extern "C"

namespace {

// ---- kernel tables: the instantiations live in the inst_*.cu units --------------------------------
DecodeKernel decode_kernel(int mb, bool cluster, int sg, bool bf, bool sym, bool a_box) {
    return bf ? decode_kernel_bf16(mb, cluster, sg, sym, a_box) : decode_kernel_f16(mb, cluster, sg, sym, a_box);
}
TileKernel tile_kernel(int mt_index, int sg, bool bf, bool sym, bool epi) {
    if (bf) return sg == 1 ? tile_kernel_bf16_sg1(mt_index, sym, epi) : sg == 2 ? tile_kernel_bf16_sg2(mt_index, sym, epi)
                                                                                : tile_kernel_bf16_sg4(mt_index, sym, epi);
    return sg == 1 ? tile_kernel_f16_sg1(mt_index, sym, epi) : sg == 2 ? tile_kernel_f16_sg2(mt_index, sym, epi)
                                                                       : tile_kernel_f16_sg4(mt_index, sym, epi);
}

// The body of every GEMM entry point; the caller holds g_mu.
int gemm_locked(const uint16_t* A, const void* Wq, const void* S, const void* Z, const uint16_t* bias, uint16_t* C,
                int M, int N, int K, int group, int split_k, int path, int flags, int act, w4a16_stream_t stream) {
    if (!flags_ok(flags)) return W4A16_ERR_SHAPE;
    const bool sym = (flags & W4A16_FLAG_SYMMETRIC) != 0, bf = (flags & W4A16_FLAG_BF16) != 0;
    if (!A || !Wq || !S || !C || (!sym && !Z)) return W4A16_ERR_NULL;
    int rc = check_weight_shape(N, K, group);
    if (rc != W4A16_OK) return rc;
    if (M < 1) return W4A16_ERR_SHAPE;
    if (act < W4A16_ACT_NONE || act > W4A16_ACT_SILU) return W4A16_ERR_SHAPE;
    if (!aligned16(A) || !aligned16(Wq) || !aligned16(S) || (!sym && !aligned16(Z)) || !aligned16(C))
        return W4A16_ERR_ALIGN;
    const int G = K / kGroup, sg = kGroup / group;
    if (split_k < 0 || split_k > G) return W4A16_ERR_SPLITK;
    if (path < W4A16_PATH_AUTO || path > W4A16_PATH_TILE) return W4A16_ERR_PATH;
    DeviceState* d = nullptr;
    if ((rc = current_device(&d)) != W4A16_OK) return rc;
    if (!d->is_sm100) return W4A16_ERR_ARCH;

    const int path_asked = path;
    path = resolve_path(M, path);
    if (split_k > 65535) return W4A16_ERR_SPLITK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const uint32_t* Zw = sym ? nullptr : static_cast<const uint32_t*>(Z);
    Epilogue epi;
    epi.bias = bias;
    epi.act = act;
    // registered workspace: [16 KiB small-M tickets][128 KiB tile tickets][partial results]
    unsigned char* ws_body = d->ws ? static_cast<unsigned char*>(d->ws) + kWsFullHeaderBytes : nullptr;
    const size_t ws_body_bytes = d->ws_bytes > kWsFullHeaderBytes ? d->ws_bytes - kWsFullHeaderBytes : 0;

    if (path == W4A16_PATH_SIMPLE) {
        if (split_k == 0) split_k = choose_split_decode(M, N, G, d->sm_count);
        if (split_k > 1 && ws_body_bytes < simple_partial_bytes(M, N, split_k)) return W4A16_ERR_WORKSPACE;
        int mchunks = (M + kSimpleMB - 1) / kSimpleMB;
        if (mchunks > 65535) return W4A16_ERR_PATH;
        float* partials = reinterpret_cast<float*>(ws_body);
        dim3 grid(N / kTileN, mchunks, split_k);
        if (bf)
            gemm_simple_kernel<true><<<grid, 64, 0, st>>>(A, static_cast<const uint32_t*>(Wq),
                                                          static_cast<const uint16_t*>(S), Zw, C, partials, M, N, K, G, sg,
                                                          split_k, epi);
        else
            gemm_simple_kernel<false><<<grid, 64, 0, st>>>(A, static_cast<const uint32_t*>(Wq),
                                                           static_cast<const uint16_t*>(S), Zw, C, partials, M, N, K, G, sg,
                                                           split_k, epi);
        if (cudaGetLastError() != cudaSuccess) return W4A16_ERR_CUDA;
        if (split_k > 1) {
            size_t MN = (size_t)M * N;
            const unsigned blocks = (unsigned)((MN + 255) / 256);
            if (bf) splitk_reduce_kernel<true><<<blocks, 256, 0, st>>>(partials, C, MN, N, split_k, epi);
            else splitk_reduce_kernel<false><<<blocks, 256, 0, st>>>(partials, C, MN, N, split_k, epi);
            if (cudaGetLastError() != cudaSuccess) return W4A16_ERR_CUDA;
        }
        return W4A16_OK;
    }

    if (path == W4A16_PATH_TILE) {
        TileGeom g = tile_geom(M, N, G, split_k, d->sm_count, d->max_smem_optin);
        if (g.stages < 2) return W4A16_ERR_PATH;
        if (g.split_k != 1) {
            if (g.tiles > kTileMaxTicketTiles) return W4A16_ERR_SPLITK;
            if (ws_body_bytes < tile_workspace_bytes(g)) return W4A16_ERR_WORKSPACE;
        }
        // (the kernel's chunk arithmetic is 32-bit)
        if ((long long)g.tiles * G >= (1ll << 31)) return W4A16_ERR_SHAPE;
        CUtensorMap tmap;
        if (!make_act_tensor_map(&tmap, A, M, K, g.mt)) return W4A16_ERR_CUDA;
        TileParams p;
        p.Wq = static_cast<const uint32_t*>(Wq);
        p.S = static_cast<const uint16_t*>(S);
        p.Z = Zw;
        p.C = C;
        p.tickets = reinterpret_cast<int*>(d->ws ? static_cast<unsigned char*>(d->ws) + kWsHeaderBytes : nullptr);
        p.ws = reinterpret_cast<float*>(ws_body);
        p.M = M; p.N = N; p.K = K; p.G = G;
        p.n_tiles = g.n_tiles;
        p.m_tiles = g.m_tiles;
        p.split_k = g.split_k;
        p.nchunks = g.nchunks;
        p.stages = g.stages;
        tile_fill_chunk_math(p);
        p.epi = epi;
        // Slices of whole tiles on CTAs of their own: the sum of the partial tiles (and with it the optional
        // bias / activation) is a second, GPU-wide kernel behind this one (kernels_basic.cuh).  Balanced
        // chunks, whose pieces belong to different tiles, keep the reduce inside the kernel.
        // Measured (us, in the kernel / second kernel): M = 256: K = 10240 / N = 4608 (four slices) 31.9 / 24.6,
        // K = 16384 / N = 4096 39.2 / 32.9, K = N = 8192 (two slices) 34.1 / 33.3; 64-row tiles are level (16.6 /
        // 16.5 at K = 11008 / N = 4096) and 32-row tiles lose the extra launch (12.9 / 13.7): from 128 rows on.
        const bool defer = g.split_k >= 2 && g.mt >= 128;
        p.defer_reduce = defer ? 1 : 0;
        const bool has_epi = !defer && (bias != nullptr || act != W4A16_ACT_NONE);
        TileKernel kern = tile_kernel(g.mt_index, sg, bf, sym, has_epi);
        bool& attr_set = d->tile_attr_set[g.mt_index][log2_sg(sg)][bf ? 1 : 0][sym ? 1 : 0][has_epi ? 1 : 0];
        if (!attr_set) {
            if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, d->max_smem_optin) !=
                cudaSuccess) {
                cudaGetLastError();
                return W4A16_ERR_CUDA;
            }
            attr_set = true;
        }
        // programmatic dependent launch: this kernel's prologue and weight prefetch may overlap the
        // tail of the previous kernel in the stream; it orders itself with griddepcontrol.wait
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(g.ctas, 1, 1);
        cfg.blockDim = dim3(tile_threads(g.mt), 1, 1);
        cfg.dynamicSmemBytes = (size_t)g.smem_bytes;
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = d->pdl_allowed(st) ? 1 : 0;
        if (cudaLaunchKernelEx(&cfg, kern, tmap, p) != cudaSuccess) {
            cudaGetLastError();
            return W4A16_ERR_CUDA;
        }
        if (defer) {
            const long long quads = (long long)g.tiles * g.mt * (kTileCols / 4);
            cudaLaunchConfig_t rcfg = {};
            rcfg.gridDim = dim3((unsigned)((quads + 255) / 256), 1, 1);
            rcfg.blockDim = dim3(256, 1, 1);
            rcfg.stream = st;
            rcfg.attrs = attr;      // always behind the GEMM kernel just launched on this stream
            rcfg.numAttrs = 1;
            const float* parts = p.ws;
            const int mt_log2 = 4 + g.mt_index;
            cudaError_t e = bf ? cudaLaunchKernelEx(&rcfg, tile_splitk_reduce_kernel<true>, parts, C, M, N, mt_log2, g.n_tiles,
                                                    g.split_k, quads, epi)
                               : cudaLaunchKernelEx(&rcfg, tile_splitk_reduce_kernel<false>, parts, C, M, N, mt_log2, g.n_tiles,
                                                    g.split_k, quads, epi);
            if (e != cudaSuccess) {
                cudaGetLastError();
                return W4A16_ERR_CUDA;
            }
        }
        return W4A16_OK;
    }

    // W4A16_PATH_DECODE
    DecodeGeom g = decode_geom(M, N, G, split_k, d->sm_count, d->cluster_ok, sg);
    if (g.mchunks > 65535 || (long)g.mchunks * (N / kTileN) > kMaxTickets) return W4A16_ERR_PATH;
    if (g.smem_bytes > d->max_smem_optin) return W4A16_ERR_PATH;
    // (the cluster exchange does not touch the workspace, but the contract stays the same for every schedule)
    if (g.split_k != 1 && ws_body_bytes < decode_partial_bytes(g)) return W4A16_ERR_WORKSPACE;
    DecodeParams p;
    p.A = A;
    p.Wq = static_cast<const uint32_t*>(Wq);
    p.S = static_cast<const uint16_t*>(S);
    p.Z = Zw;
    p.C = C;
    p.ws = reinterpret_cast<float*>(ws_body);
    p.tickets = static_cast<int*>(d->ws);
    p.M = M; p.N = N; p.K = K; p.G = G; p.T = N / kTileN;
    p.split_k = g.split_k;
    p.nchunks = g.nchunks;
    p.stages = g.stages;
    p.stage_bytes = g.stage_bytes;
    p.prefetch = g.prefetch;
    decode_fill_chunk_math(p);
    p.epi = epi;
    CUtensorMap tmap_a;
    if (g.a_box) {
        if (!make_decode_tensor_map(&tmap_a, A, M, K, g.mb)) return W4A16_ERR_CUDA;
    } else {
        memset(&tmap_a, 0, sizeof(tmap_a));
    }
    DecodeKernel kern = decode_kernel(g.mb, g.cluster, sg, bf, sym, g.a_box);
    bool& attr_set = d->decode_attr_set[g.mb][g.cluster ? 1 : 0][log2_sg(sg)][bf ? 1 : 0][sym ? 1 : 0][g.a_box ? 1 : 0];
    if (!attr_set) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, d->max_smem_optin) !=
            cudaSuccess) {
            cudaGetLastError();
            return W4A16_ERR_CUDA;
        }
        attr_set = true;
    }
    // programmatic dependent launch (see the tile path above): prologue and weight prefetch may overlap
    // the tail of the previous kernel in the stream
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(g.ctas, g.mchunks, 1);
    cfg.blockDim = dim3(kDecThreads, 1, 1);
    cfg.dynamicSmemBytes = (size_t)g.smem_bytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    int n_attr = 0;
    if (g.cluster) {   // the split_k CTAs of a column tile are one cluster (consecutive blockIdx.x)
        attr[n_attr].id = cudaLaunchAttributeClusterDimension;
        attr[n_attr].val.clusterDim.x = (unsigned)g.split_k;
        attr[n_attr].val.clusterDim.y = 1;
        attr[n_attr].val.clusterDim.z = 1;
        ++n_attr;
    }
    if (d->pdl_allowed(st)) {
        attr[n_attr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n_attr].val.programmaticStreamSerializationAllowed = 1;
        ++n_attr;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n_attr;
    if (cudaLaunchKernelEx(&cfg, kern, tmap_a, p) != cudaSuccess) {
        cudaGetLastError();
        if (g.cluster) {
            // the device would not place the clusters: from now on the workspace exchange (and the path
            // rule that goes with it), starting with this call
            d->cluster_ok = false;
            return gemm_locked(A, Wq, S, Z, bias, C, M, N, K, group, split_k, path_asked, flags, act, stream);
        }
        return W4A16_ERR_CUDA;
    }
    return W4A16_OK;
}
}  // namespace

extern "C" {

int w4a16_gemm_fmt(const uint16_t* A, const void* Wq, const void* S, const void* Z, const uint16_t* bias, uint16_t* C,
                   int M, int N, int K, int group, int split_k, int path, int flags, int act, w4a16_stream_t stream) {
    std::lock_guard<std::mutex> lock(g_mu);
    if (bias != nullptr && (reinterpret_cast<uintptr_t>(bias) & 1u)) return W4A16_ERR_ALIGN;
    return gemm_locked(A, Wq, S, Z, bias, C, M, N, K, group, split_k, path, flags, act, stream);
}

int w4a16_gemm_ex(const uint16_t* A, const void* Wq, const void* S, const void* Z, uint16_t* C, int M, int N, int K,
                  int group, int split_k, int path, w4a16_stream_t stream) {
    std::lock_guard<std::mutex> lock(g_mu);
    if (!Z) return W4A16_ERR_NULL;
    return gemm_locked(A, Wq, S, Z, nullptr, C, M, N, K, group, split_k, path, 0, W4A16_ACT_NONE, stream);
}

int w4a16_gemm(const uint16_t* A, const void* Wq, const void* S, const void* Z, uint16_t* C, int M, int N, int K,
               int group, int split_k, w4a16_stream_t stream) {
    return w4a16_gemm_ex(A, Wq, S, Z, C, M, N, K, group, split_k, W4A16_PATH_AUTO, stream);
}

int w4a16_gemm_host(const uint16_t* A_host, uint16_t* A_dev, const void* Wq, const void* S, const void* Z,
                    uint16_t* C_dev, uint16_t* C_host, int M, int N, int K, int group, int split_k,
                    w4a16_stream_t stream) {
    if (!A_host || !A_dev || !C_dev || !C_host) return W4A16_ERR_NULL;
    if (M < 1 || K < 1 || N < 1) return W4A16_ERR_SHAPE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(A_dev, A_host, (size_t)M * K * 2, cudaMemcpyHostToDevice, st) != cudaSuccess) {
        cudaGetLastError();
        return W4A16_ERR_CUDA;
    }
    // Page-locked host memory that the device can address takes the result straight from the kernel's stores
    // (each element of C is written once, by whoever finishes its sum): one copy and one runtime call less.
    // Anything else goes through C_dev and a copy.
    uint16_t* c_direct = nullptr;
    {
        cudaPointerAttributes attr;
        if (cudaPointerGetAttributes(&attr, C_host) == cudaSuccess) {
            if (attr.type == cudaMemoryTypeHost && attr.devicePointer != nullptr && aligned16(attr.devicePointer))
                c_direct = static_cast<uint16_t*>(attr.devicePointer);
        } else {
            cudaGetLastError();
        }
    }
    int rc = w4a16_gemm(A_dev, Wq, S, Z, c_direct ? c_direct : C_dev, M, N, K, group, split_k, stream);
    if (rc != W4A16_OK) return rc;
    if (!c_direct && cudaMemcpyAsync(C_host, C_dev, (size_t)M * N * 2, cudaMemcpyDeviceToHost, st) != cudaSuccess) {
        cudaGetLastError();
        return W4A16_ERR_CUDA;
    }
    return W4A16_OK;
}

int w4a16_gemm_static_ws(const uint16_t* A, const void* Wq, const void* S, const void* Z, uint16_t* C, int M, int N,
                         int K, int group, int split_k, w4a16_stream_t stream) {
    std::lock_guard<std::mutex> lock(g_mu);
    if (!A || !Wq || !S || !Z || !C) return W4A16_ERR_NULL;
    int rc = check_weight_shape(N, K, group);
    if (rc != W4A16_OK) return rc;
    if (M < 1) return W4A16_ERR_SHAPE;
    if (!aligned16(A) || !aligned16(Wq) || !aligned16(S) || !aligned16(Z) || !aligned16(C)) return W4A16_ERR_ALIGN;
    const int G = K / kGroup, sg = kGroup / group;
    if (split_k < 0 || split_k > G) return W4A16_ERR_SPLITK;
    DeviceState* d = nullptr;
    if ((rc = current_device(&d)) != W4A16_OK) return rc;
    if (!d->is_sm100) return W4A16_ERR_ARCH;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return W4A16_ERR_CUDA;

    const DecodeGeom g = decode_geom(M, N, G, split_k, d->sm_count, false, sg);   // no clusters here: this entry point keeps the path it was built with
    if (g.mchunks > 65535 || (long)g.mchunks * (N / kTileN) > kMaxTickets) return W4A16_ERR_PATH;
    if (g.smem_bytes > d->max_smem_optin) return W4A16_ERR_PATH;
    // the whole scratch need of this shape must fit the built-in array, or nothing is launched (a schedule of
    // whole tiles, split_k == 1, leaves no partial tiles and draws no tickets: it needs none)
    if (g.split_k != 1 && kWsHeaderBytes + decode_partial_bytes(g) > (size_t)W4A16_STATIC_WS_BYTES)
        return W4A16_ERR_WORKSPACE;

    // first call on this device: resolve the array's device address (this device is current)
    if (g_static_ws_addr[dev] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_ws) != cudaSuccess || p == nullptr) {
            cudaGetLastError();
            return W4A16_ERR_CUDA;
        }
        g_static_ws_addr[dev] = static_cast<unsigned char*>(p);
    }
    unsigned char* ws = g_static_ws_addr[dev];
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the array keeps whatever the previous call left; the ticket counters must start at zero
    if (cudaMemsetAsync(ws, 0, kWsHeaderBytes, st) != cudaSuccess) {
        cudaGetLastError();
        return W4A16_ERR_CUDA;
    }
    DecodeParams p;
    p.A = A;
    p.Wq = static_cast<const uint32_t*>(Wq);
    p.S = static_cast<const uint16_t*>(S);
    p.Z = static_cast<const uint32_t*>(Z);
    p.C = C;
    p.ws = reinterpret_cast<float*>(ws + kWsHeaderBytes);
    p.tickets = reinterpret_cast<int*>(ws);
    p.M = M; p.N = N; p.K = K; p.G = G; p.T = N / kTileN;
    p.split_k = g.split_k;
    p.nchunks = g.nchunks;
    p.stages = g.stages;
    p.stage_bytes = g.stage_bytes;
    p.prefetch = g.prefetch;
    decode_fill_chunk_math(p);
    CUtensorMap tmap_a;
    if (g.a_box) {
        if (!make_decode_tensor_map(&tmap_a, A, M, K, g.mb)) return W4A16_ERR_CUDA;
    } else {
        memset(&tmap_a, 0, sizeof(tmap_a));
    }
    p.epi.bias = nullptr;
    p.epi.act = kActNone;
    DecodeKernel kern = decode_kernel(g.mb, false, sg, false, false, g.a_box);
    bool& attr_set = d->decode_attr_set[g.mb][0][log2_sg(sg)][0][0][g.a_box ? 1 : 0];
    if (!attr_set) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, d->max_smem_optin) !=
            cudaSuccess) {
            cudaGetLastError();
            return W4A16_ERR_CUDA;
        }
        attr_set = true;
    }
    kern<<<dim3(g.ctas, g.mchunks, 1), kDecThreads, g.smem_bytes, st>>>(tmap_a, p);
    return cudaGetLastError() == cudaSuccess ? W4A16_OK : W4A16_ERR_CUDA;
}

int w4a16_selftest_wait_timeout(unsigned limit_us, w4a16_stream_t stream) {
    std::lock_guard<std::mutex> lock(g_mu);
    if (limit_us < 1 || limit_us > 100000) return W4A16_ERR_SHAPE;
    DeviceState* d = nullptr;
    int rc = current_device(&d);
    if (rc != W4A16_OK) return rc;
    if (!d->is_sm100) return W4A16_ERR_ARCH;
    wait_timeout_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>((unsigned long long)limit_us * 1000ull,
                                                                               nullptr);
    return cudaGetLastError() == cudaSuccess ? W4A16_OK : W4A16_ERR_CUDA;
}

int w4a16_device_status(int* status_out) {
    std::lock_guard<std::mutex> lock(g_mu);
    if (!status_out) return W4A16_ERR_NULL;
    if (cudaDeviceSynchronize() != cudaSuccess) {
        cudaGetLastError();
        return W4A16_ERR_CUDA;
    }
    // every translation unit that holds kernels has a status word of its own
    const int words[] = {status_take_this_unit(),     status_take_decode_f16(),   status_take_decode_bf16(),
                         status_take_tile_f16_sg1(),  status_take_tile_f16_sg2(), status_take_tile_f16_sg4(),
                         status_take_tile_bf16_sg1(), status_take_tile_bf16_sg2(), status_take_tile_bf16_sg4()};
    int v = 0;
    for (int w : words) {
        if (w < 0) return W4A16_ERR_CUDA;
        v |= w;
    }
    *status_out = v;
    if (v != 0) {
        // a kernel that gave up returned before it drew its tickets: the counters of the registered
        // workspace may be non-zero, and the next call would take a tile for complete too early
        DeviceState* d = nullptr;
        if (current_device(&d) == W4A16_OK && d->ws != nullptr &&
            (cudaMemset(d->ws, 0, kWsFullHeaderBytes) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess)) {
            cudaGetLastError();
            return W4A16_ERR_CUDA;
        }
    }
    return v == 0 ? W4A16_OK : W4A16_ERR_DEVICE_STATUS;
}

}  // extern "C"
