/*
 * CPU oracle for the W4A16 matrix multiplication  C = A . Dequant(W),
 * Dequant(W) = s (W - z)  (paper Eq. 2, Section "Method").
 *
 * TEST INFRASTRUCTURE ONLY.  Plain, slow, written from the definition: no
 * blocking, fusion, Split-K or reordering.  It shares no code with the CUDA
 * path and is never on the product path; only the tests, the smoke check and
 * the benchmark's cpu-baseline leg may load it.
 *
 * Conventions (the paper leaves them open; these are the readings used):
 *   - W is unsigned INT4, 0..15, with an integer zero point z in 0..15.
 *   - INT4 values are stored 8 per 32-bit word along K (storage packing,
 *     Section 2.2): word Wq[kk, n] of the row-major array [K/8, N] holds
 *     q[8*kk + i, n] in bits 4i .. 4i+3.
 *   - s and z are per (group, column): S f16 [K/group, N], Z u8 [K/group, N].
 *   - "Dequantize to FP16" (Algorithm 1, Phase 1): the multiplicand is the
 *     FP16-rounded weight  w16 = fp16_rn((q - z) * s).  (q - z) is exact and
 *     its product with an FP16 s is exact in double, so there is exactly one
 *     rounding (nearest-even, subnormals kept).
 *   - C_ref = sum_k A[m,k] * w16[k,n] accumulated in FP64 (Eq. 2); it is NOT
 *     rounded to FP16 -- the tests apply the tolerance to double(C_gpu) - C_ref.
 *   - Phase 3 (sum of the S partial results, then FP32 -> FP16) only changes the
 *     summation order, so the definition above is the oracle for every split.
 *
 * Every function below is pinned by tests/test_oracle_*.py against something
 * other than itself (IEEE-754 encodings, numpy float16, exact rational
 * arithmetic on tiny shapes, the exact-integer closed form, invariants).
 */
#include <stdint.h>
#include <stddef.h>
#include <string.h>
#include <math.h>
#include <stdlib.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ---- IEEE-754 binary16 <-> binary32/64, written from the format definition ---- */

/* binary16: 1 sign, 5 exponent (bias 15), 10 fraction bits. */
float orc_f16_to_f32(uint16_t h)
{
    uint32_t sign = (uint32_t)(h >> 15) & 1u;
    int      e    = (int)((h >> 10) & 0x1Fu);
    uint32_t f    = (uint32_t)(h & 0x3FFu);
    double v;
    if (e == 0) {
        v = ldexp((double)f, -24);               /* subnormal or zero: f * 2^-24 */
    } else if (e == 31) {
        v = f ? NAN : INFINITY;
    } else {
        v = ldexp((double)(1024u + f), e - 25);  /* (1 + f/1024) * 2^(e-15) */
    }
    return (float)(sign ? -v : v);
}

/* Round a double to the nearest binary16, ties to even; overflow -> Inf. */
uint16_t orc_f64_to_f16_rn(double x)
{
    uint16_t sign = 0;
    if (isnan(x)) return 0x7E00u;
    if (signbit(x)) { sign = 0x8000u; x = -x; }
    if (isinf(x)) return (uint16_t)(sign | 0x7C00u);
    if (x == 0.0) return sign;

    int ex;
    (void)frexp(x, &ex);           /* x = m * 2^ex, m in [0.5, 1) -> x in [2^(ex-1), 2^ex) */
    int e = ex - 1;                /* floor(log2 x) */
    /* spacing of binary16 values around x: 2^(e-10) for normals, 2^-24 below 2^-14 */
    int ulp_exp = (e < -14) ? -24 : (e - 10);
    double scaled = ldexp(x, -ulp_exp);          /* exact: power-of-two scaling */
    double r = nearbyint(scaled);                /* default rounding mode: nearest-even */
    /* r is an integer count of ulps; rebuild the encoding from the value r * 2^ulp_exp */
    if (r == 0.0) return sign;
    double v = ldexp(r, ulp_exp);
    if (v >= 65520.0) return (uint16_t)(sign | 0x7C00u);   /* 65520 = halfway past max, rounds to Inf */
    if (v > 65504.0)  v = 65504.0;                          /* cannot happen; guard */
    /* encode v exactly (v is representable) */
    int ev;
    (void)frexp(v, &ev);
    int fe = ev - 1;
    if (fe < -14) {
        uint32_t frac = (uint32_t)ldexp(v, 24);             /* subnormal: v / 2^-24 */
        return (uint16_t)(sign | frac);
    } else {
        uint32_t mant = (uint32_t)ldexp(v, 10 - fe);        /* in [1024, 2048) */
        return (uint16_t)(sign | ((uint32_t)(fe + 15) << 10) | (mant - 1024u));
    }
}

uint16_t orc_f32_to_f16_rn(float x) { return orc_f64_to_f16_rn((double)x); }

/* ---- bfloat16 <-> binary32/64 (Section 1 names BF16 beside FP16 as the dequantization target) ----
 * bfloat16: 1 sign, 8 exponent (bias 127), 7 fraction bits: the upper half of a binary32. */
float orc_bf16_to_f32(uint16_t h)
{
    uint32_t sign = (uint32_t)(h >> 15) & 1u;
    int      e    = (int)((h >> 7) & 0xFFu);
    uint32_t f    = (uint32_t)(h & 0x7Fu);
    double v;
    if (e == 0) {
        v = ldexp((double)f, -133);              /* subnormal or zero: f * 2^-133 */
    } else if (e == 255) {
        v = f ? NAN : INFINITY;
    } else {
        v = ldexp((double)(128u + f), e - 134);  /* (1 + f/128) * 2^(e-127) */
    }
    return (float)(sign ? -v : v);
}

/* Round a double to the nearest bfloat16, ties to even; overflow -> Inf. */
uint16_t orc_f64_to_bf16_rn(double x)
{
    uint16_t sign = 0;
    if (isnan(x)) return 0x7FC0u;
    if (signbit(x)) { sign = 0x8000u; x = -x; }
    if (isinf(x)) return (uint16_t)(sign | 0x7F80u);
    if (x == 0.0) return sign;
    int ex;
    (void)frexp(x, &ex);
    int e = ex - 1;                               /* floor(log2 x) */
    /* spacing of bfloat16 values around x: 2^(e-7) for normals, 2^-133 below 2^-126 */
    int ulp_exp = (e < -126) ? -133 : (e - 7);
    double r = nearbyint(ldexp(x, -ulp_exp));     /* integer count of ulps, ties to even */
    if (r == 0.0) return sign;
    double v = ldexp(r, ulp_exp);
    if (v >= ldexp(1.0, 128)) return (uint16_t)(sign | 0x7F80u);   /* rounded past the largest finite value */
    int ev;
    (void)frexp(v, &ev);
    int fe = ev - 1;
    if (fe < -126) {
        uint32_t frac = (uint32_t)ldexp(v, 133);
        return (uint16_t)(sign | frac);
    } else {
        uint32_t mant = (uint32_t)ldexp(v, 7 - fe);            /* in [128, 256) */
        return (uint16_t)(sign | ((uint32_t)(fe + 127) << 7) | (mant - 128u));
    }
}

/* The 16-bit format of activations, scales, dequantized weights and output: 0 = FP16, 1 = BF16. */
static inline double orc_widen(uint16_t bits, int bf16)
{
    return (double)(bf16 ? orc_bf16_to_f32(bits) : orc_f16_to_f32(bits));
}
static inline uint16_t orc_round16(double x, int bf16)
{
    return bf16 ? orc_f64_to_bf16_rn(x) : orc_f64_to_f16_rn(x);
}

/* ---- unpack (Section 2.2: INT4 values packed into INT32 words) ---- */

/* q[k, n] for all k < K, n < N as one byte each, row-major [K, N]. */
void orc_unpack(const uint32_t *Wq, int K, int N, uint8_t *q)
{
    for (int k = 0; k < K; ++k)
        for (int n = 0; n < N; ++n) {
            uint32_t word = Wq[(size_t)(k / 8) * N + n];
            q[(size_t)k * N + n] = (uint8_t)((word >> (4 * (k % 8))) & 15u);
        }
}

static inline int orc_q_at(const uint32_t *Wq, int N, int k, int n)
{
    return (int)((Wq[(size_t)(k / 8) * N + n] >> (4 * (k % 8))) & 15u);
}

/* ---- Dequant(W) = s (W - z), rounded once to FP16 (Eq. 2; Algorithm 1, Phase 1) ---- */

static inline uint16_t orc_dequant_one(int q, int z, uint16_t s_bits, int bf16)
{
    double s = orc_widen(s_bits, bf16);
    return orc_round16((double)(q - z) * s, bf16);   /* subtract first, multiply once, round once */
}

/* W16[k, n], 16-bit patterns (FP16, or BF16 when bf16 != 0), row-major [K, N]. */
void orc_dequant_fmt(const uint32_t *Wq, const uint16_t *S, const uint8_t *Z,
                     int K, int N, int group, int bf16, uint16_t *W16)
{
    #pragma omp parallel for schedule(static)
    for (int k = 0; k < K; ++k) {
        int g = k / group;
        for (int n = 0; n < N; ++n)
            W16[(size_t)k * N + n] =
                orc_dequant_one(orc_q_at(Wq, N, k, n), Z[(size_t)g * N + n], S[(size_t)g * N + n], bf16);
    }
}

void orc_dequant(const uint32_t *Wq, const uint16_t *S, const uint8_t *Z,
                 int K, int N, int group, uint16_t *W16)
{
    orc_dequant_fmt(Wq, S, Z, K, N, group, 0, W16);
}

/* ---- C = A . Dequant(W) in FP64 (Eq. 2) ---- */

/* A: FP16 bits [M, K] row-major.  C_ref: double [M, N] row-major.
 * Only columns n0 <= n < n1 are written, and only k0 <= k < k1 is summed
 * (n0 = 0, n1 = N, k0 = 0, k1 = K for the whole product).  Column n of
 * Dequant(W) is formed once (FP16-rounded, then widened) and every row of A is
 * multiplied into it. */
void orc_gemm_kslice_cols_fmt(const uint16_t *A, const uint32_t *Wq, const uint16_t *S, const uint8_t *Z,
                              int M, int N, int K, int group, int k0, int k1, int n0, int n1, int bf16,
                              double *C_ref)
{
    #pragma omp parallel
    {
        double *wcol = (double *)malloc(sizeof(double) * (size_t)K);
        #pragma omp for schedule(static)
        for (int n = n0; n < n1; ++n) {
            for (int k = k0; k < k1; ++k) {
                int g = k / group;
                uint16_t w16 = orc_dequant_one(orc_q_at(Wq, N, k, n),
                                               Z[(size_t)g * N + n], S[(size_t)g * N + n], bf16);
                wcol[k] = orc_widen(w16, bf16);
            }
            for (int m = 0; m < M; ++m) {
                double acc = 0.0;
                for (int k = k0; k < k1; ++k)
                    acc += orc_widen(A[(size_t)m * K + k], bf16) * wcol[k];
                C_ref[(size_t)m * N + n] = acc;
            }
        }
        free(wcol);
    }
}

void orc_gemm_kslice_cols(const uint16_t *A, const uint32_t *Wq, const uint16_t *S, const uint8_t *Z,
                          int M, int N, int K, int group, int k0, int k1, int n0, int n1,
                          double *C_ref)
{
    orc_gemm_kslice_cols_fmt(A, Wq, S, Z, M, N, K, group, k0, k1, n0, n1, 0, C_ref);
}

/* The whole product in the chosen 16-bit format (0 = FP16, 1 = BF16). */
void orc_gemm_fmt(const uint16_t *A, const uint32_t *Wq, const uint16_t *S, const uint8_t *Z,
                  int M, int N, int K, int group, int bf16, double *C_ref)
{
    orc_gemm_kslice_cols_fmt(A, Wq, S, Z, M, N, K, group, 0, K, 0, N, bf16, C_ref);
}

void orc_gemm_cols(const uint16_t *A, const uint32_t *Wq, const uint16_t *S, const uint8_t *Z,
                   int M, int N, int K, int group, int n0, int n1, double *C_ref)
{
    orc_gemm_kslice_cols(A, Wq, S, Z, M, N, K, group, 0, K, n0, n1, C_ref);
}

void orc_gemm(const uint16_t *A, const uint32_t *Wq, const uint16_t *S, const uint8_t *Z,
              int M, int N, int K, int group, double *C_ref)
{
    orc_gemm_cols(A, Wq, S, Z, M, N, K, group, 0, N, C_ref);
}

/* The K-slice [k0, k1) alone: the partial result C_i of Phase 2 for one split. */
void orc_gemm_kslice(const uint16_t *A, const uint32_t *Wq, const uint16_t *S, const uint8_t *Z,
                     int M, int N, int K, int group, int k0, int k1, double *C_part)
{
    orc_gemm_kslice_cols(A, Wq, S, Z, M, N, K, group, k0, k1, 0, N, C_part);
}

/* ---- exact case: integer A, power-of-two scales ----
 * With A[m,k] a small integer (given as int8) and s[g,n] = 2^E[g,n]
 * (E an int8 exponent, -14 <= E <= 15), every product and every partial sum of
 * Eq. 2 is an integer multiple of 2^Emin, so the sum has ONE exact value; the
 * FP32 -> FP16 cast of Phase 3 then gives fp16_rn(exact).  Accumulates in
 * int64 and returns FP16 bits [M, N].  Returns nonzero if Emin..Emax spans more
 * than 30 binary places (would not fit the int64 scaling used here).
 */
int orc_gemm_int_fmt(const int8_t *A, const uint32_t *Wq, const int8_t *E, const uint8_t *Z,
                     int M, int N, int K, int group, int bf16, uint16_t *C16)
{
    int G = K / group;
    int emin = 127, emax = -128;
    for (size_t i = 0; i < (size_t)G * N; ++i) {
        if (E[i] < emin) emin = E[i];
        if (E[i] > emax) emax = E[i];
    }
    if (emax - emin > 30) return 1;
    for (int m = 0; m < M; ++m)
        for (int n = 0; n < N; ++n) {
            int64_t total = 0;                                  /* in units of 2^emin */
            for (int g = 0; g < G; ++g) {
                int64_t part = 0;
                int z = Z[(size_t)g * N + n];
                for (int k = g * group; k < (g + 1) * group; ++k)
                    part += (int64_t)A[(size_t)m * K + k] * (int64_t)(orc_q_at(Wq, N, k, n) - z);
                total += part * ((int64_t)1 << (E[(size_t)g * N + n] - emin));
            }
            C16[(size_t)m * N + n] = orc_round16(ldexp((double)total, emin), bf16);
        }
    return 0;
}

int orc_gemm_int(const int8_t *A, const uint32_t *Wq, const int8_t *E, const uint8_t *Z,
                 int M, int N, int K, int group, uint16_t *C16)
{
    return orc_gemm_int_fmt(A, Wq, E, Z, M, N, K, group, 0, C16);
}

/* ---- the step before the path: the affine quantizer of Eq. 1,  x_q = round(x / s) + z ----
 * The paper gives the formula and says that symmetric quantization fixes z; how s and z are chosen, the
 * rounding of ties and the clamp are open.  Readings used here, per group of `group` consecutive k of one
 * column n (the granularity of s and z on the GEMM side):
 *   asymmetric: s = (max - min) / 15 over the group, rounded to the 16-bit format (this stored value is
 *               the s of every later step); z = clamp(round(-min / s), 0, 15);
 *   symmetric:  s = max|x| / 7, z = 8 (codes q - 8 in -8 .. 7);
 *   a group whose s would be zero (all values equal, or all zero) or not finite gets s = 1;
 *   q = clamp(round(x / s) + z, 0, 15); round = to nearest, ties to even.
 * Floating point decides integers here, so the precision is part of the definition: every operation is
 * a single IEEE binary32 operation (subtract, divide, round-to-integer) in the order written; x and s enter
 * as the exact values of their 16-bit patterns.
 */
static inline float orc_group_scale(float num, float den, int bf16)
{
    float s32 = num / den;
    uint16_t b = orc_round16((double)s32, bf16);
    float s = (float)orc_widen(b, bf16);
    if (!(s > 0.0f) || isinf(s)) s = 1.0f;
    return s;
}

void orc_quantize(const uint16_t *W16, int K, int N, int group, int symmetric, int bf16,
                  uint32_t *Wq, uint16_t *S, uint8_t *Z)
{
    int G = K / group;
    memset(Wq, 0, sizeof(uint32_t) * (size_t)(K / 8) * N);
    for (int g = 0; g < G; ++g)
        for (int n = 0; n < N; ++n) {
            float lo = INFINITY, hi = -INFINITY, amax = 0.0f;
            for (int k = g * group; k < (g + 1) * group; ++k) {
                float x = (float)orc_widen(W16[(size_t)k * N + n], bf16);
                if (x < lo) lo = x;
                if (x > hi) hi = x;
                if (fabsf(x) > amax) amax = fabsf(x);
            }
            float s;
            int z;
            if (symmetric) {
                s = orc_group_scale(amax, 7.0f, bf16);
                z = 8;
            } else {
                s = orc_group_scale(hi - lo, 15.0f, bf16);
                float zf = nearbyintf(-lo / s);
                z = zf < 0.0f ? 0 : zf > 15.0f ? 15 : (int)zf;
            }
            S[(size_t)g * N + n] = orc_round16((double)s, bf16);   /* s is representable: exact */
            Z[(size_t)g * N + n] = (uint8_t)z;
            for (int k = g * group; k < (g + 1) * group; ++k) {
                float x = (float)orc_widen(W16[(size_t)k * N + n], bf16);
                float r = nearbyintf(x / s) + (float)z;
                int q = r < 0.0f ? 0 : r > 15.0f ? 15 : (int)r;
                Wq[(size_t)(k / 8) * N + n] |= (uint32_t)q << (4 * (k % 8));
            }
        }
}

int orc_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
