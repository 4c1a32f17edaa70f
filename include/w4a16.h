/*
 * w4a16.h -- C ABI of the B200 (sm_100a) W4A16 matrix multiplication library.
 *
 *     C[M,N] = A[M,K] . Dequant(W)[K,N],   Dequant(W) = s (W - z)        (paper Eq. 2)
 *
 * A is FP16, W is unsigned INT4 (0..15) with one FP16 scale s and one integer zero
 * point z (0..15) per group of `group` consecutive k (128, 64 or 32) and per column n,
 * accumulation is FP32 and C is FP16 (Algorithm 1: dequantize, Split-K multiply,
 * reduce + FP32->FP16 cast).  The *_fmt entry points add the format variants the paper
 * names without fixing them: symmetric quantization (Eq. 1 with the zero point fixed, here
 * z = 8 for the unsigned nibbles, i.e. q - 8 in -8 .. 7, and no Z buffer) and BF16 instead of
 * FP16 for activations, scales, dequantized weights and output (Section 1).
 *
 * General rules
 *   - Every pointer is a DEVICE pointer owned by the caller unless a parameter says
 *     "host".  The library allocates no device memory, keeps no reference to a buffer
 *     after the work it enqueued has completed, and never frees anything.
 *   - Calls enqueue work on `stream` (a cudaStream_t passed as void*; NULL = the
 *     default stream) and return without waiting.  Argument errors are detected on the
 *     host, returned at once, and launch nothing.
 *   - Return value: W4A16_OK (0) or a negative W4A16_ERR_* code; w4a16_strerror()
 *     names it.  Nothing is printed, nothing throws, nothing exits.
 *   - FP16 values cross the boundary as their 16-bit patterns (uint16_t).
 *   - Device code exists for sm_100a only; on any other device the launching calls
 *     return W4A16_ERR_ARCH.
 *
 * Raw layout (what w4a16_pack consumes; storage packing of 4-bit values into 32-bit words,
 * Section 2.2):
 *   Wq_raw  uint32 [K/8, N] row-major; bits 4i..4i+3 of Wq_raw[kk, n] hold q[8 kk + i, n]
 *   S_raw   FP16   [K/group, N] row-major
 *   Z_raw   uint8  [K/group, N] row-major, one zero point (0..15) per byte
 * Packed layout (what the kernels consume): opaque; sizes from w4a16_packed_*_bytes.
 *
 * Preconditions shared by pack / dequant / gemm:  group in {32, 64, 128}, K > 0,
 * K % 128 == 0, N > 0, N % 64 == 0; all buffers 16-byte aligned.  Violations ->
 * W4A16_ERR_SHAPE / W4A16_ERR_ALIGN / W4A16_ERR_NULL.
 */
#ifndef W4A16_H_
#define W4A16_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef void *w4a16_stream_t; /* a cudaStream_t; NULL = default stream */

enum {
    W4A16_OK = 0,
    W4A16_ERR_NULL = -1,          /* a required pointer is NULL */
    W4A16_ERR_SHAPE = -2,         /* M, N, K or group outside the supported set */
    W4A16_ERR_ALIGN = -3,         /* a buffer is not 16-byte aligned */
    W4A16_ERR_SPLITK = -4,        /* split_k < 0 or > K/128 */
    W4A16_ERR_WORKSPACE = -5,     /* split_k > 1 needs more workspace than was set */
    W4A16_ERR_CUDA = -6,          /* a CUDA runtime call failed (launch, attribute, copy) */
    W4A16_ERR_ARCH = -7,          /* current device is not sm_100 */
    W4A16_ERR_DEVICE_STATUS = -8, /* a kernel gave up on a bounded wait; see w4a16_device_status */
    W4A16_ERR_PATH = -9           /* requested kernel path cannot run this shape */
};

/* Kernel selection for w4a16_gemm_ex.  AUTO picks by shape. */
enum {
    W4A16_PATH_AUTO = 0,
    W4A16_PATH_SIMPLE = 1, /* plain FP32-FMA kernel, any M; two-kernel Split-K reduce */
    W4A16_PATH_DECODE = 2, /* small-M bandwidth-bound kernel (M <= 64): TMA bulk staging,
                              in-register unpack, warp-level tensor-core MMA */
    W4A16_PATH_TILE = 3    /* tcgen05 / TMEM tile kernel, any M (batch tiles of 16 .. 256 rows) */
};

/* Format options of the *_fmt entry points (bit flags). */
enum {
    W4A16_FLAG_SYMMETRIC = 1, /* zero point 8 for every weight; Z pointers are ignored and may be NULL */
    W4A16_FLAG_BF16 = 2       /* A, S, the dequantized weights and C are BF16 instead of FP16 */
};

/* Optional step fused into the final cast of w4a16_gemm_fmt (not part of Algorithm 1). */
enum {
    W4A16_ACT_NONE = 0,
    W4A16_ACT_RELU = 1, /* max(x, 0) */
    W4A16_ACT_SILU = 2  /* x / (1 + exp(-x)) */
};

const char *w4a16_strerror(int code);

/* Sizes in bytes of the three packed buffers for a [K, N] weight matrix (0 if the shape
 * is not supported).  The packed form holds exactly the information of the raw form:
 * K*N/2 bytes of nibbles, 2 bytes per scale, 4 bits per zero point. */
size_t w4a16_packed_wq_bytes(int N, int K, int group);
size_t w4a16_packed_s_bytes(int N, int K, int group);
size_t w4a16_packed_z_bytes(int N, int K, int group);

/* Split-K (Algorithm 1, Phase 2/3) keeps FP32 partial results C_i in a caller-owned
 * device workspace.  w4a16_workspace_bytes: bytes needed by w4a16_gemm for this shape
 * and split_k (split_k == 0 means "whatever w4a16_choose_split_k picks"); 0 when no
 * workspace is needed.
 * w4a16_set_workspace: registers the buffer for the CURRENT device (one per device, per
 * process; replaces the previous one; dev_ptr == NULL, bytes == 0 unregisters).  The
 * buffer must be 256-byte aligned and at least W4A16_WORKSPACE_HEADER_BYTES long, stays
 * owned by the caller and must outlive every gemm call enqueued while it is registered.  The
 * call zeroes that header (the kernels' ticket counters) on the default stream and waits.  gemm calls that need the workspace and overlap on
 * the GPU (different streams) race on it; serialise them or use split_k = 1. */
#define W4A16_WORKSPACE_HEADER_BYTES (16384u + 131072u)
size_t w4a16_workspace_bytes(int M, int N, int K, int group, int split_k);
int w4a16_set_workspace(void *dev_ptr, size_t bytes);

/* The split factor S the library picks for a shape when split_k == 0 (the paper takes S
 * as an input and gives no rule; Section 4.1 says when it pays: K >> N).  Always a value
 * w4a16_gemm accepts; >= 1.  `path` as in w4a16_gemm_ex. */
int w4a16_choose_split_k(int M, int N, int K, int group);
int w4a16_choose_split_k_ex(int M, int N, int K, int group, int path);
/* The kernel path (W4A16_PATH_*) w4a16_gemm takes for a shape, or a negative error code. */
int w4a16_choose_path(int M, int N, int K, int group);

/* Offline reorder of the raw nibbles, scales and zero points into the packed layout
 * (pure data movement, a bijection; Section 2.2 storage packing).  Reads the three raw
 * device arrays, writes the three packed device buffers (sizes above). */
int w4a16_pack(const uint32_t *Wq_raw, const uint16_t *S_raw, const uint8_t *Z_raw,
               void *Wq, void *S, void *Z, int N, int K, int group, w4a16_stream_t stream);

/* Algorithm 1, Phase 1 as a standalone operation: W16[k, n] = fp16_rn((q - z) * s),
 * one rounding to nearest-even, subnormals kept.  Wq, S, Z are PACKED buffers.
 * W16: FP16 [K, N] row-major, fully overwritten. */
int w4a16_dequant(const void *Wq, const void *S, const void *Z, uint16_t *W16,
                  int N, int K, int group, w4a16_stream_t stream);

/* Eq. 2 / Algorithm 1: C = A . Dequant(W), FP32 accumulation, Split-K over `split_k`
 * slices of whole groups (slice sizes differ by at most one group, the first
 * (K/group) mod split_k slices get the extra one), partial results summed in ascending
 * slice order in FP32, one FP32->FP16 rounding (nearest-even) at the end.
 *   A   FP16 [M, K] row-major (K contiguous), M >= 1
 *   Wq, S, Z   packed buffers from w4a16_pack
 *   C   FP16 [M, N] row-major, fully overwritten (no beta)
 *   split_k   0 = automatic, else 1 <= split_k <= K/128: slices are whole blocks of 128 k,
 *             i.e. whole groups for every supported group size (some paths cap it lower
 *             and return W4A16_ERR_SPLITK beyond their cap)
 * Results are bit-identical from run to run for fixed arguments (with split_k == 0 the schedule,
 * and with it the order of the FP32 sums, is the library's choice for this entry point and device;
 * it changes once, for good, if the device refuses a thread-block-cluster launch).  If the chosen
 * split needs workspace and too little is registered: W4A16_ERR_WORKSPACE.
 * Ordering: A, C and the workspace are touched in stream order.  The packed buffers Wq, S, Z
 * may be read (prefetched) while the previous kernel of the stream is still running, so
 * they must not be written by in-flight work other than a w4a16_pack enqueued earlier on the
 * same stream (the library makes the first GEMM launch on each stream after a pack a fully
 * ordered one; a pack on ANOTHER stream needs the caller's own event or synchronisation before
 * the GEMM, as for any cross-stream dependency); pack weights once, at load. */
int w4a16_gemm(const uint16_t *A, const void *Wq, const void *S, const void *Z, uint16_t *C,
               int M, int N, int K, int group, int split_k, w4a16_stream_t stream);

/* Same operation with the kernel path forced (W4A16_PATH_*); for tests and benchmarks.
 * W4A16_ERR_PATH if that path does not support the shape. */
int w4a16_gemm_ex(const uint16_t *A, const void *Wq, const void *S, const void *Z, uint16_t *C,
                  int M, int N, int K, int group, int split_k, int path, w4a16_stream_t stream);

/* The same three operations with the format options above (flags = 0 and act = W4A16_ACT_NONE,
 * bias = NULL give exactly w4a16_pack / w4a16_dequant / w4a16_gemm_ex).
 *   W4A16_FLAG_SYMMETRIC   Eq. 1's symmetric case: every zero point is 8; Z_raw / Z are not read
 *                          and no Z traffic exists (pass NULL).
 *   W4A16_FLAG_BF16        S_raw / S, A, W16 and C hold BF16 bit patterns; the dequantized weight
 *                          is bf16_rn((q - z) * s), accumulation stays FP32, one FP32->BF16
 *                          rounding at the end.  (pack only moves 16-bit scales: the flag does
 *                          not change it.)
 *   bias   NULL, or [N] values in C's 16-bit format added to the FP32 sum before `act` and the
 *          final rounding:  C[m, n] = rn16(act(sum + bias[n])).
 * Everything else (layouts, split_k, path, ordering, error codes) is as documented above. */
int w4a16_pack_fmt(const uint32_t *Wq_raw, const uint16_t *S_raw, const uint8_t *Z_raw,
                   void *Wq, void *S, void *Z, int N, int K, int group, int flags,
                   w4a16_stream_t stream);
int w4a16_dequant_fmt(const void *Wq, const void *S, const void *Z, uint16_t *W16,
                      int N, int K, int group, int flags, w4a16_stream_t stream);
int w4a16_gemm_fmt(const uint16_t *A, const void *Wq, const void *S, const void *Z,
                   const uint16_t *bias, uint16_t *C, int M, int N, int K, int group,
                   int split_k, int path, int flags, int act, w4a16_stream_t stream);

/* The step before the path: the affine quantizer of Eq. 1, x_q = round(x / s) + z, applied per group
 * of `group` consecutive k and per column to 16-bit weights W16 [K, N] row-major (FP16, or BF16 with
 * W4A16_FLAG_BF16), writing the RAW layout that w4a16_pack[_fmt] consumes.  The paper gives the formula
 * only; this library fixes the rest as follows.
 *   asymmetric  s = (max - min) / 15 over the group, rounded to the 16-bit format;
 *               z = clamp(round(-min / s), 0, 15)
 *   symmetric (W4A16_FLAG_SYMMETRIC)  s = max|x| / 7, z = 8; Z_raw is not written and may be NULL
 *   s == 0 or not finite -> s = 1;  q = clamp(round(x / s) + z, 0, 15);  round = nearest, ties to even;
 *   every operation is a single IEEE binary32 operation, so the codes are reproducible bit for bit.
 * Offline (weights are quantized once); not part of the timed path. */
int w4a16_quantize(const uint16_t *W16, uint32_t *Wq_raw, uint16_t *S_raw, uint8_t *Z_raw,
                   int N, int K, int group, int flags, w4a16_stream_t stream);

/* End-to-end form of w4a16_gemm for callers whose activations live in HOST memory:
 * copies A_host (FP16 [M, K], ideally pinned) into the caller's device staging buffer
 * A_dev, runs w4a16_gemm into the device staging buffer C_dev, and copies the result
 * into C_host (FP16 [M, N]); all three steps are enqueued on `stream` in order.  If
 * C_host is page-locked host memory that the device can address (cudaHostAlloc /
 * cudaHostRegister, 16-byte aligned), the kernel stores the result there itself: the
 * copy is skipped and C_dev is not written.  The host buffers must stay valid until the
 * stream has run them.  Weights stay resident on the device (they are the model's
 * parameters, packed once). */
int w4a16_gemm_host(const uint16_t *A_host, uint16_t *A_dev, const void *Wq, const void *S,
                    const void *Z, uint16_t *C_dev, uint16_t *C_host, int M, int N, int K,
                    int group, int split_k, w4a16_stream_t stream);

/* No counterpart in the paper: an extra entry point for callers that must not allocate.
 *
 * Some hosts of this library cannot hand it a workspace: an inference runtime that sizes all
 * of its device memory at start-up and forbids cudaMalloc afterwards (an allocation stalls the
 * whole device), a plug-in that runs inside someone else's memory pool, a control loop with a
 * latency bound, or code on a path where the allocator may not be entered at all.  For them
 * this call computes the same product as w4a16_gemm on the small-M kernel (the one whose
 * Split-K keeps FP32 partial tiles and ticket counters in scratch memory), but takes that
 * scratch from an array of W4A16_STATIC_WS_BYTES bytes built into the library's device image
 * instead of the buffer registered with w4a16_set_workspace.  It calls no cudaMalloc, no
 * cudaFree and no allocating library routine; A, Wq, S, Z and C are still the caller's.
 *
 *   - Cost: every GPU on which the library is loaded holds the W4A16_STATIC_WS_BYTES until the
 *     process exits, whether or not this call is ever made.
 *   - Limit: a shape / split_k whose scratch need (16 KiB of counters + the partial tiles, the
 *     same amount w4a16_workspace_bytes reports for the small-M kernel) exceeds the array is
 *     rejected with W4A16_ERR_WORKSPACE and nothing is launched.  A schedule of whole tiles
 *     (split_k = 1, or split_k = 0 where the library picks whole tiles) needs no scratch and
 *     always fits; every M <= 16 with split_k = 0 fits; large explicit split_k on wide N may not.
 *   - The first call on each device looks up the array's device address (one
 *     cudaGetSymbolAddress with that device current) and sets a kernel attribute; make that
 *     first call outside any stream capture.  Later calls only enqueue work.
 *   - All calls on a device share the one array and it keeps the previous call's contents.
 *     Each call first clears the counter block with a cudaMemsetAsync on `stream`, then
 *     launches the kernel.  Two calls that overlap on the GPU (different streams, or this call
 *     from two threads) race on the array: keep them ordered.
 *   - Arguments, preconditions, result and error codes are otherwise those of w4a16_gemm. */
#define W4A16_STATIC_WS_BYTES (4u * 1024u * 1024u + 16384u)
int w4a16_gemm_static_ws(const uint16_t *A, const void *Wq, const void *S, const void *Z,
                         uint16_t *C, int M, int N, int K, int group, int split_k,
                         w4a16_stream_t stream);

/* Every wait inside the kernels on a barrier or on another CTA has a limit (two seconds): a
 * wait that runs out records a code in a status word on the device, the kernel releases what
 * it holds and returns.  (The one instruction that can block without a limit is the tensor-
 * memory allocation of the tile kernel; it cannot wait on another CTA of this library because
 * the kernel asks for more than half of an SM's shared memory, so two of its CTAs never share
 * an SM, and each frees its columns before it returns.)
 * w4a16_device_status synchronises the current device, copies the word to *status_out
 * (0 = no kernel gave up since the last call; bit 0 = a barrier wait ran out) and clears it.
 * If it was nonzero the call also zeroes the ticket counters of the registered workspace (a
 * kernel that gave up may have left them mid-count) and returns W4A16_ERR_DEVICE_STATUS; the
 * output of the GEMM calls since the previous status check is then undefined, later calls
 * work normally. */
int w4a16_device_status(int *status_out);

/* Diagnostic for the path above, no counterpart in the paper: enqueues a one-warp kernel whose
 * only action is a bounded wait, limit `limit_us` microseconds (1 .. 100000), on a barrier that
 * nothing ever arrives on.  The wait runs out, the kernel records the code and returns; the next
 * w4a16_device_status reports it.  Nothing faults and the context stays usable. */
int w4a16_selftest_wait_timeout(unsigned limit_us, w4a16_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* W4A16_H_ */
