/*
 * W2A8 reference ("oracle") -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, scalar CPU statement of what the W2A8 path computes:
 * 2-bit weight codes x int8 activations -> exact int32 per-group sums ->
 * scaled fp32 outputs.  It exists so that the CUDA library can be checked
 * against something that can be verified by eye; it shares no code, header,
 * table or helper with the CUDA sources and must never be called from the
 * product path.  Only the tests, the smoke check and the CPU-baseline /
 * reference legs of the benchmark may build or call it.
 *
 * Conventions (GEMM naming, not the paper's): M = tokens, N = output
 * channels, K = contraction length, g = group length along K with one fp32
 * weight scale per (channel, group).  The paper names the weight matrix A
 * (its M x K), the activations B (its N x K) and the result C.
 *
 * What each routine follows:
 *   ref_pack / ref_unpack : the idea of Sec. II-B / II-C (Fig. 1, left): store
 *       the frozen 2-bit codes ahead of time so that one shift+mask of a
 *       32-bit word yields four int8 lanes that are consecutive along K,
 *       i.e. already in the order an int8 dot-product instruction wants.
 *       The concrete bit layout ("W2P") is this build's own and is written
 *       out below; the paper's AVX2 layout is not reproduced.
 *   ref_quantize : Sec. II-D: scale from the abs-max of the quantisation
 *       granule (here: one token = all K entries); every entry times the
 *       inverse of that scale, rounded to nearest even, as int8.
 *   ref_partials : Sec. II-C microkernel result: int32 = sum of
 *       int8 activation x (2-bit weight as int8), exact.
 *   ref_gemm : Sec. II-D dequantisation: int32 -> float, times the product
 *       of activation scale and weight scale; with K-groups the weight scale
 *       is applied per group before summing.
 *   ref_half_to_float / ref_float_to_bf16 / ref_gemm_h : the recipe of the
 *       end-to-end ternary section (groups of 128 along K, weight scales
 *       stored in 16 bits; the 16-bit format is read as IEEE binary16, the
 *       type the direct-conversion listing of Sec. II names for its scale):
 *       the same sums as ref_gemm with each scale first widened exactly to
 *       fp32, and an optional bf16 result (round to nearest even of the
 *       fp32 result).
 *   ref_gemm_a16 : the alternative kernel of Sec. II ("Alternative
 *       implementation"): the 2-bit weights are used as 16-bit values against
 *       16-bit activations, with no activation quantisation and no
 *       dequantisation step: y = sum_k x[k] * (value[k] * scale[group of k]),
 *       here with x in bf16 and the sum written group by group.
 *
 * Parity pins: every routine here is pinned by tests that do not reuse this
 * code (hand-written golden words, exhaustive exact-rational evaluation of
 * the quantiser, brute force / closed forms for the integer sums, exact
 * rationals for the outputs).  The quantiser's rounding rule and scale
 * formula are fixed by this build's reading of the paper, not by a printed
 * value in the paper.
 *
 * Build: gcc -O2 -ffp-contract=off -fopenmp -shared -fPIC (no fast-math).
 * OpenMP only splits independent output channels / tokens between threads;
 * it does not change any result.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int ref_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ---------------------------------------------------------------- layout */
/*
 * W2P layout of one output channel (row) of K codes, K a multiple of 64.
 *
 *  - A "group slice" is 64 consecutive k.  A "block" is up to four
 *    consecutive slices: block b covers k in [256 b, 256 b + 64 R) where
 *    R = min(4, (K - 256 b) / 64) is the number of slices it holds.
 *  - A 32-bit word holds 16 consecutive k.  Inside block b, the word that
 *    holds k = 256 b + 64 s + 16 t + l  (slice s < R, quarter t < 4, l < 16)
 *    is stored at word index  16 b + t * R + s  of the row.  So in a full
 *    block the 16-byte unit number t carries quarter t of each of the four
 *    slices; a block with R = 1 is in natural order.
 *  - Inside the word, code l sits at bit 8 * (l mod 4) + 2 * (l div 4):
 *    byte (l mod 4), 2-bit slot (l div 4).  Hence (word >> 2 j) & 0x03030303
 *    is four consecutive-k codes (l = 4 j .. 4 j + 3), one per byte.
 *  - Rows follow one another; a row is K / 16 words, the matrix K * N / 4
 *    bytes.
 */
static size_t w2p_word_index(int K, int k) {
    int b = k / 256;
    int rem = K - 256 * b;
    int R = rem >= 256 ? 4 : rem / 64;
    int kb = k % 256;
    int s = kb / 64;
    int t = (kb % 64) / 16;
    return (size_t)16 * b + (size_t)t * R + s;
}

static int w2p_bit_offset(int k) {
    int l = k % 16;
    return 8 * (l % 4) + 2 * (l / 4);
}

/* codes[N][K] with values 0..3 (higher bits ignored) -> packed[N][K/16] */
void ref_pack(const uint8_t *codes, int N, int K, uint32_t *packed) {
    size_t words = (size_t)K / 16;
    memset(packed, 0, (size_t)N * words * sizeof(uint32_t));
    for (int n = 0; n < N; ++n)
        for (int k = 0; k < K; ++k) {
            uint32_t c = codes[(size_t)n * K + k] & 3u;
            packed[(size_t)n * words + w2p_word_index(K, k)] |= c << w2p_bit_offset(k);
        }
}

void ref_unpack(const uint32_t *packed, int N, int K, uint8_t *codes) {
    size_t words = (size_t)K / 16;
    for (int n = 0; n < N; ++n)
        for (int k = 0; k < K; ++k) {
            uint32_t w = packed[(size_t)n * words + w2p_word_index(K, k)];
            codes[(size_t)n * K + k] = (uint8_t)((w >> w2p_bit_offset(k)) & 3u);
        }
}

/* ------------------------------------------------------------- quantiser */
static float bf16_to_float(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/*
 * Per-token symmetric abs-max quantisation of bf16 activations to int8.
 * Every fp32 operation below is one IEEE-754 round-to-nearest-even
 * operation (compile with -ffp-contract=off):
 *   amax = max_k |x|;  s = amax / 127;  inv = 1 / s;  a = rne(x * inv),
 * clamped to [-127, 127].  A row whose amax is 0, or so small that inv is
 * not finite, quantises to all zeros with scale 0.
 * x: [M][K] bf16 bit patterns;  a: [M][K];  a_scale: [M].
 */
void ref_quantize(const uint16_t *x, int M, int K, int8_t *a, float *a_scale) {
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        const uint16_t *xr = x + (size_t)m * K;
        int8_t *ar = a + (size_t)m * K;
        float amax = 0.0f;
        for (int k = 0; k < K; ++k) {
            float v = fabsf(bf16_to_float(xr[k]));
            if (v > amax) amax = v;
        }
        volatile float s = amax / 127.0f;
        volatile float inv = 1.0f / s;
        if (!(amax > 0.0f) || !isfinite(inv)) {
            memset(ar, 0, (size_t)K);
            a_scale[m] = 0.0f;
            continue;
        }
        a_scale[m] = s;
        for (int k = 0; k < K; ++k) {
            volatile float t = bf16_to_float(xr[k]) * inv;
            float r = nearbyintf(t); /* default rounding mode: ties to even */
            if (r > 127.0f) r = 127.0f;
            if (r < -127.0f) r = -127.0f;
            ar[k] = (int8_t)r;
        }
    }
}

/* ------------------------------------------------------- integer partials */
/*
 * P[m][n][gi] = sum over k in group gi of a[m][k] * (q[n][k] - 2), exact.
 * a: [M][K] int8; codes: [N][K] (0..3); P: [M][N][K/g] int32.
 */
void ref_partials(const int8_t *a, const uint8_t *codes, int M, int N, int K, int g,
                  int32_t *P) {
    int G = K / g;
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n)
        for (int m = 0; m < M; ++m)
            for (int gi = 0; gi < G; ++gi) {
                int32_t acc = 0;
                for (int k = gi * g; k < (gi + 1) * g; ++k)
                    acc += (int32_t)a[(size_t)m * K + k] *
                           ((int32_t)(codes[(size_t)n * K + k] & 3) - 2);
                P[((size_t)m * N + n) * G + gi] = acc;
            }
}

/* ---------------------------------------------------------------- outputs */
/*
 * y[m][n] = fp32( a_scale[m] * sum_gi w_scale[n][gi] * P[m][n][gi] ),
 * the sum and products carried in double in index order.
 * w_scale: [N][K/g] fp32; y: [M][N] fp32.
 */
void ref_gemm(const int8_t *a, const float *a_scale, const uint8_t *codes,
              const float *w_scale, int M, int N, int K, int g, float *y) {
    int G = K / g;
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n)
        for (int m = 0; m < M; ++m) {
            double acc = 0.0;
            for (int gi = 0; gi < G; ++gi) {
                int32_t p = 0;
                for (int k = gi * g; k < (gi + 1) * g; ++k)
                    p += (int32_t)a[(size_t)m * K + k] *
                         ((int32_t)(codes[(size_t)n * K + k] & 3) - 2);
                acc += (double)w_scale[(size_t)n * G + gi] * (double)p;
            }
            y[(size_t)m * N + n] = (float)((double)a_scale[m] * acc);
        }
}

/* ------------------------------------------------- 16-bit scales / outputs */
/*
 * IEEE binary16 bit pattern -> its value, field by field: 1 sign bit, 5
 * exponent bits (bias 15), 10 fraction bits; exponent 0 = subnormal
 * (fraction * 2^-24), exponent 31 = infinity / NaN.  Every binary16 value is
 * a float, so the result is exact.
 */
float ref_half_to_float(uint16_t h) {
    int sign = (h >> 15) & 1, e = (h >> 10) & 31, frac = h & 1023;
    double v;
    if (e == 0)       v = ldexp((double)frac, -24);
    else if (e == 31) v = frac ? (double)NAN : (double)INFINITY;
    else              v = ldexp((double)(1024 + frac), e - 25);
    return (float)(sign ? -v : v);
}

/*
 * float -> bf16 bit pattern (the upper 16 bits of a float whose lower 16 bits
 * are zero), round to nearest, ties to the even 16-bit pattern; overflow goes
 * to infinity as in IEEE; NaN stays NaN (quiet bit set).  Written as a
 * comparison of the discarded half with one half unit, not as a bias trick.
 */
uint16_t ref_float_to_bf16(float f) {
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u);
    uint32_t keep = u >> 16, rest = u & 0xffffu;
    if (rest > 0x8000u || (rest == 0x8000u && (keep & 1u))) keep += 1u;   /* may carry into the exponent */
    return (uint16_t)keep;
}

/*
 * ref_gemm with w_scale given as binary16 bit patterns [N][K/g].  y32 (fp32
 * [M][N]) is always written; y16 (bf16 bit patterns [M][N]) when not NULL is
 * the rounding of the same fp32 values.
 */
void ref_gemm_h(const int8_t *a, const float *a_scale, const uint8_t *codes,
                const uint16_t *w_scale_h, int M, int N, int K, int g, float *y32, uint16_t *y16) {
    int G = K / g;
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n)
        for (int m = 0; m < M; ++m) {
            double acc = 0.0;
            for (int gi = 0; gi < G; ++gi) {
                int32_t p = 0;
                for (int k = gi * g; k < (gi + 1) * g; ++k)
                    p += (int32_t)a[(size_t)m * K + k] *
                         ((int32_t)(codes[(size_t)n * K + k] & 3) - 2);
                acc += (double)ref_half_to_float(w_scale_h[(size_t)n * G + gi]) * (double)p;
            }
            float r = (float)((double)a_scale[m] * acc);
            y32[(size_t)m * N + n] = r;
            if (y16) y16[(size_t)m * N + n] = ref_float_to_bf16(r);
        }
}

/* ------------------------------------------- 16-bit activations, no quantiser */
/*
 * y[m][n] = fp32( sum_gi w_scale[n][gi] * sum_{k in gi} x[m][k] * (q[n][k] - 2) ),
 * x given as bf16 bit patterns, everything carried in double in index order
 * (every product x * (q - 2) is exact in double, and so is its product with
 * nothing else until the scale).
 * x: [M][K] bf16 bits; codes: [N][K]; w_scale: [N][K/g] fp32; y: [M][N] fp32.
 */
void ref_gemm_a16(const uint16_t *x, const uint8_t *codes, const float *w_scale,
                  int M, int N, int K, int g, float *y) {
    int G = K / g;
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n)
        for (int m = 0; m < M; ++m) {
            double acc = 0.0;
            for (int gi = 0; gi < G; ++gi) {
                double p = 0.0;
                for (int k = gi * g; k < (gi + 1) * g; ++k)
                    p += (double)bf16_to_float(x[(size_t)m * K + k]) *
                         (double)((int)(codes[(size_t)n * K + k] & 3) - 2);
                acc += (double)w_scale[(size_t)n * G + gi] * p;
            }
            y[(size_t)m * N + n] = (float)acc;
        }
}
