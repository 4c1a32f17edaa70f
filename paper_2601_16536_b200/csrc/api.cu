// C ABI of the library (declared in include/w4a16.h): argument validation, per-shape
// kernel and Split-K selection, launches.  Every step of the computation runs in the
// kernels included below; this file only marshals arguments.
#include "w4a16.h"

#include <cuda_runtime.h>

#include "common.cuh"
#include "kernels_basic.cuh"
#include "kernel_decode.cuh"

using namespace w4a16;

namespace {

constexpr int kMaxDevices = 64;
constexpr size_t kWsHeaderBytes = 4096;  // zeroed control words ahead of the FP32 partials

struct DeviceState {
    bool probed = false;
    bool is_sm100 = false;
    int sm_count = 148;
    int max_smem_optin = 0;
    void* ws = nullptr;
    size_t ws_bytes = 0;
    bool decode_attr_set[3] = {false, false, false};
};
DeviceState g_dev[kMaxDevices];

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
    if (group != kGroup) return W4A16_ERR_SHAPE;
    if (K <= 0 || N <= 0 || K % kGroup != 0 || N % kTileN != 0) return W4A16_ERR_SHAPE;
    return W4A16_OK;
}

int sm_count_or_default() {
    DeviceState* d = nullptr;
    if (current_device(&d) == W4A16_OK) return d->sm_count;
    return 148;
}

// ---- decode-path launch geometry ------------------------------------------------
int decode_mb(int M) { return M <= 8 ? 1 : 2; }

struct DecodeGeom {
    int mb, stages, sz_bytes, smem_bytes, ctas_per_sm;
};

DecodeGeom decode_geom(int M, int G, int split_k) {
    DecodeGeom g;
    g.mb = decode_mb(M);
    int max_ng = (G + split_k - 1) / split_k;
    g.sz_bytes = ((max_ng * (kSBlockHalves * 2 + kZBlockWords * 4)) + 127) / 128 * 128;
    int stage = decode_stage_bytes(8 * g.mb);
    int n_iter = (max_ng + kDecWarps - 1) / kDecWarps;
    // two CTAs per SM when the ring fits twice in 227 KiB, else one
    int budget2 = (227 * 1024) / 2 - 1024 - 128 - g.sz_bytes;
    int budget1 = 227 * 1024 - 1024 - 128 - g.sz_bytes;
    int st = budget2 / stage;
    g.ctas_per_sm = 2;
    if (st < 3) {
        st = budget1 / stage;
        g.ctas_per_sm = 1;
    }
    if (st > 6) st = 6;
    if (st > n_iter) st = n_iter;
    if (st < 1) st = 1;
    g.stages = st;
    g.smem_bytes = 128 + g.sz_bytes + st * stage;
    return g;
}

int choose_split_decode(int M, int N, int G, int sms) {
    // Model: CTAs = tiles * m_chunks * S run in waves of (sms * resident CTAs); a CTA's time
    // is its groups plus a fixed start-up/reduce cost (in units of one group's time).
    int mb = decode_mb(M);
    long tiles = (long)(N / kTileN) * ((M + 8 * mb - 1) / (8 * mb));
    int best = 1;
    double best_cost = 1e30;
    for (int s = 1; s <= 16; s *= 2) {
        if (s > G) break;
        if (s > 1 && G / s < 2) break;
        DecodeGeom g = decode_geom(M, G, s);
        long slots = (long)sms * g.ctas_per_sm;
        long ctas = tiles * s;
        long waves = (ctas + slots - 1) / slots;
        double per_cta = (double)((G + s - 1) / s) + 6.0;
        // fewer resident CTAs than slots still share the same HBM: scale by occupancy of the last wave
        double cost = (double)waves * per_cta + (s > 1 ? 2.0 + 0.5 * s : 0.0);
        if (ctas < slots) cost = per_cta * 1.0 + (s > 1 ? 2.0 + 0.5 * s : 0.0) + (double)(slots - ctas) / slots * 8.0;
        if (cost < best_cost - 1e-9) {
            best_cost = cost;
            best = s;
        }
    }
    return best;
}

int resolve_path(int M, int path) {
    if (path == W4A16_PATH_AUTO) return W4A16_PATH_DECODE;
    return path;
}

size_t partial_bytes(int M, int N, int split_k) {
    size_t b = (size_t)split_k * (size_t)M * (size_t)N * sizeof(float);
    return (b + 255) / 256 * 256;
}

}  // namespace

// =====================================================================================
extern "C" {

const char* w4a16_strerror(int code) {
    switch (code) {
        case W4A16_OK: return "ok";
        case W4A16_ERR_NULL: return "null pointer argument";
        case W4A16_ERR_SHAPE: return "unsupported shape (need group == 128, K % 128 == 0, N % 64 == 0, M >= 1)";
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
size_t w4a16_packed_z_bytes(int N, int K, int group) {
    if (check_weight_shape(N, K, group) != W4A16_OK) return 0;
    return (size_t)(K / group) * (size_t)N / 2;
}

int w4a16_choose_split_k_ex(int M, int N, int K, int group, int path) {
    if (check_weight_shape(N, K, group) != W4A16_OK || M < 1) return 1;
    int G = K / group;
    switch (resolve_path(M, path)) {
        case W4A16_PATH_DECODE: return choose_split_decode(M, N, G, sm_count_or_default());
        default: return 1;
    }
}
int w4a16_choose_split_k(int M, int N, int K, int group) {
    return w4a16_choose_split_k_ex(M, N, K, group, W4A16_PATH_AUTO);
}

size_t w4a16_workspace_bytes(int M, int N, int K, int group, int split_k) {
    if (check_weight_shape(N, K, group) != W4A16_OK || M < 1 || split_k < 0) return 0;
    if (split_k == 0) split_k = w4a16_choose_split_k(M, N, K, group);
    if (split_k <= 1) return 0;
    return kWsHeaderBytes + partial_bytes(M, N, split_k);
}

int w4a16_set_workspace(void* dev_ptr, size_t bytes) {
    DeviceState* d = nullptr;
    int rc = current_device(&d);
    if (rc != W4A16_OK) return rc;
    if (dev_ptr == nullptr || bytes == 0) {
        d->ws = nullptr;
        d->ws_bytes = 0;
        return W4A16_OK;
    }
    if ((reinterpret_cast<uintptr_t>(dev_ptr) & 255u) != 0) return W4A16_ERR_ALIGN;
    if (bytes < kWsHeaderBytes) return W4A16_ERR_WORKSPACE;
    if (cudaMemset(dev_ptr, 0, kWsHeaderBytes) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) {
        cudaGetLastError();
        return W4A16_ERR_CUDA;
    }
    d->ws = dev_ptr;
    d->ws_bytes = bytes;
    return W4A16_OK;
}

int w4a16_pack(const uint32_t* Wq_raw, const uint16_t* S_raw, const uint8_t* Z_raw, void* Wq, void* S, void* Z,
               int N, int K, int group, w4a16_stream_t stream) {
    if (!Wq_raw || !S_raw || !Z_raw || !Wq || !S || !Z) return W4A16_ERR_NULL;
    int rc = check_weight_shape(N, K, group);
    if (rc != W4A16_OK) return rc;
    if (!aligned16(Wq_raw) || !aligned16(S_raw) || !aligned16(Z_raw) || !aligned16(Wq) || !aligned16(S) ||
        !aligned16(Z))
        return W4A16_ERR_ALIGN;
    DeviceState* d = nullptr;
    if ((rc = current_device(&d)) != W4A16_OK) return rc;
    if (!d->is_sm100) return W4A16_ERR_ARCH;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int G = K / group;
    size_t words = (size_t)K * N / 8, sc = (size_t)G * N, zw = (size_t)G * N / 8;
    pack_wq_kernel<<<(unsigned)((words + 255) / 256), 256, 0, st>>>(Wq_raw, static_cast<uint32_t*>(Wq), N, G, words);
    pack_s_kernel<<<(unsigned)((sc + 255) / 256), 256, 0, st>>>(S_raw, static_cast<uint16_t*>(S), N, G, sc);
    pack_z_kernel<<<(unsigned)((zw + 255) / 256), 256, 0, st>>>(Z_raw, static_cast<uint32_t*>(Z), N, G, zw);
    return cudaGetLastError() == cudaSuccess ? W4A16_OK : W4A16_ERR_CUDA;
}

int w4a16_dequant(const void* Wq, const void* S, const void* Z, uint16_t* W16, int N, int K, int group,
                  w4a16_stream_t stream) {
    if (!Wq || !S || !Z || !W16) return W4A16_ERR_NULL;
    int rc = check_weight_shape(N, K, group);
    if (rc != W4A16_OK) return rc;
    if (!aligned16(Wq) || !aligned16(S) || !aligned16(Z) || !aligned16(W16)) return W4A16_ERR_ALIGN;
    DeviceState* d = nullptr;
    if ((rc = current_device(&d)) != W4A16_OK) return rc;
    if (!d->is_sm100) return W4A16_ERR_ARCH;
    size_t words = (size_t)K * N / 8;
    dequant_kernel<<<(unsigned)((words + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint32_t*>(Wq), static_cast<const __half*>(S), static_cast<const uint32_t*>(Z),
        reinterpret_cast<__half*>(W16), N, K / group, words);
    return cudaGetLastError() == cudaSuccess ? W4A16_OK : W4A16_ERR_CUDA;
}

int w4a16_gemm_ex(const uint16_t* A, const void* Wq, const void* S, const void* Z, uint16_t* C, int M, int N, int K,
                  int group, int split_k, int path, w4a16_stream_t stream) {
    if (!A || !Wq || !S || !Z || !C) return W4A16_ERR_NULL;
    int rc = check_weight_shape(N, K, group);
    if (rc != W4A16_OK) return rc;
    if (M < 1) return W4A16_ERR_SHAPE;
    if (!aligned16(A) || !aligned16(Wq) || !aligned16(S) || !aligned16(Z) || !aligned16(C)) return W4A16_ERR_ALIGN;
    const int G = K / group;
    if (split_k < 0 || split_k > G) return W4A16_ERR_SPLITK;
    if (path < W4A16_PATH_AUTO || path > W4A16_PATH_TILE) return W4A16_ERR_PATH;
    DeviceState* d = nullptr;
    if ((rc = current_device(&d)) != W4A16_OK) return rc;
    if (!d->is_sm100) return W4A16_ERR_ARCH;

    path = resolve_path(M, path);
    if (path == W4A16_PATH_TILE) return W4A16_ERR_PATH;
    if (split_k == 0) split_k = w4a16_choose_split_k_ex(M, N, K, group, path);
    if (split_k > 65535) return W4A16_ERR_SPLITK;

    float* partials = nullptr;
    if (split_k > 1) {
        size_t need = kWsHeaderBytes + partial_bytes(M, N, split_k);
        if (d->ws == nullptr || d->ws_bytes < need) return W4A16_ERR_WORKSPACE;
        partials = reinterpret_cast<float*>(static_cast<unsigned char*>(d->ws) + kWsHeaderBytes);
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const __half* Ah = reinterpret_cast<const __half*>(A);
    __half* Ch = reinterpret_cast<__half*>(C);

    if (path == W4A16_PATH_SIMPLE) {
        int mchunks = (M + kSimpleMB - 1) / kSimpleMB;
        if (mchunks > 65535) return W4A16_ERR_PATH;
        dim3 grid(N / kTileN, mchunks, split_k);
        gemm_simple_kernel<<<grid, 64, 0, st>>>(Ah, static_cast<const uint32_t*>(Wq), static_cast<const __half*>(S),
                                                static_cast<const uint32_t*>(Z), Ch, partials, M, N, K, G, split_k);
    } else {  // W4A16_PATH_DECODE
        DecodeGeom g = decode_geom(M, G, split_k);
        int mchunks = (M + 8 * g.mb - 1) / (8 * g.mb);
        if (mchunks > 65535) return W4A16_ERR_PATH;
        if (g.smem_bytes > d->max_smem_optin) return W4A16_ERR_PATH;
        DecodeParams p;
        p.A = Ah;
        p.Wq = static_cast<const uint32_t*>(Wq);
        p.S = static_cast<const __half*>(S);
        p.Z = static_cast<const uint32_t*>(Z);
        p.C = Ch;
        p.ws = partials;
        p.M = M; p.N = N; p.K = K; p.G = G;
        p.split_k = split_k;
        p.stages = g.stages;
        p.sz_bytes = g.sz_bytes;
        auto kern = (g.mb == 1) ? gemm_decode_kernel<1> : gemm_decode_kernel<2>;
        if (!d->decode_attr_set[g.mb]) {
            if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, d->max_smem_optin) !=
                cudaSuccess) {
                cudaGetLastError();
                return W4A16_ERR_CUDA;
            }
            d->decode_attr_set[g.mb] = true;
        }
        dim3 grid(N / kTileN, split_k, mchunks);
        kern<<<grid, kDecThreads, g.smem_bytes, st>>>(p);
    }
    if (cudaGetLastError() != cudaSuccess) return W4A16_ERR_CUDA;
    if (split_k > 1) {
        size_t MN = (size_t)M * N;
        splitk_reduce_kernel<<<(unsigned)((MN + 255) / 256), 256, 0, st>>>(partials, Ch, MN, split_k);
        if (cudaGetLastError() != cudaSuccess) return W4A16_ERR_CUDA;
    }
    return W4A16_OK;
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
    int rc = w4a16_gemm(A_dev, Wq, S, Z, C_dev, M, N, K, group, split_k, stream);
    if (rc != W4A16_OK) return rc;
    if (cudaMemcpyAsync(C_host, C_dev, (size_t)M * N * 2, cudaMemcpyDeviceToHost, st) != cudaSuccess) {
        cudaGetLastError();
        return W4A16_ERR_CUDA;
    }
    return W4A16_OK;
}

int w4a16_device_status(int* status_out) {
    if (!status_out) return W4A16_ERR_NULL;
    int v = 0, zero = 0;
    if (cudaDeviceSynchronize() != cudaSuccess ||
        cudaMemcpyFromSymbol(&v, g_status_word, sizeof(int)) != cudaSuccess ||
        cudaMemcpyToSymbol(g_status_word, &zero, sizeof(int)) != cudaSuccess) {
        cudaGetLastError();
        return W4A16_ERR_CUDA;
    }
    *status_out = v;
    return v == 0 ? W4A16_OK : W4A16_ERR_DEVICE_STATUS;
}

}  // extern "C"
