/*
 * FGMP oracle -- TEST INFRASTRUCTURE, not the product.
 *
 * A plain, slow CPU statement of what the FGMP linear layer computes, written from
 * the paper's definitions.  It shares no code, tables or headers with the CUDA
 * library and must never be called from a product path.
 *
 * What follows what:
 *   - number formats: NVFP4 = 16-element blocks of FP4 (E2M1) with one FP8 (E4M3)
 *     microscale; FP8 (E4M3) without microscaling as the high precision; one metadata
 *     bit per block (Section 4, first paragraph; Section 5.1).
 *   - quantization error Delta_p v = Q_p(v) - v                              (Eq. 2)
 *   - block impact score  I  = sum_i g_i^2 (Delta v_i)^2                      (Eq. 6)
 *                          I' = sum_i g_i^2 (Delta_{pl} v_i - Delta_{ph} v_i)^2 (Eq. 7-8)
 *   - local threshold: the top fraction R of one tensor's blocks is kept in FP8 (Eq. 9)
 *   - sensitivity-weighted clipping: brute force over the FP8 scale values   (Eq. 11)
 *   - dynamic-max scaling for activations                  (Section 3.3, last sentence)
 *   - activation rule: FP8 iff the weighted error sum is greater than the threshold
 *     (Section 4.2)
 *   - mixed dot product with FP32-or-better accumulation (Section 4.1): here fp64.
 *
 * Rounding is done by exhaustive search over the representable grid (15 E2M1 values,
 * 253 finite E4M3 values): nearest value, ties to the even code, magnitudes above
 * the largest finite value saturate, the sign of the input is kept even when the
 * magnitude rounds to zero.  No bit tricks.
 *
 * Single-precision steps are single IEEE operations (compile with
 * -ffp-contract=off, no fast-math).  The sequence is, per block of 16 values v_i
 * with tensor scale s4 (FP32) and the FP8 tensor scale s8 (FP32): given on its own
 * (Section 5.1: FP8 blocks have no microscale, only a per-tensor scale), or, when
 * the argument is 0, tied to s4 as s8 = s4 * 2^ratio:
 *     amax = max |v_i|;  k6 = 1 / (6 * s4);  c0 = E4M3(amax * k6)     (dynamic max)
 *     d = e4m3val(c) * s4;  inv = 1 / d;  code_i = E2M1(v_i * inv);  dq4_i = e2m1val(code_i) * d
 *     inv8 = 1 / s8;  code8_i = E4M3(v_i * inv8);  dq8_i = e4m3val(code8_i) * s8
 *     mode 0: e_i = v_i - dq4_i      mode 1: e_i = dq4_i - dq8_i
 *     score = sum_{i=0..15, in order} (f_i * e_i) * e_i
 *
 * Parity status: every function here is pinned by tests (format tables, exhaustive
 * rounding against an independent midpoint routine and a library cast, brute-force
 * clip search in fp64, fraction invariant, memory closed form, tau extremes, fp64
 * library matmul).  Unpinned: the effect of the method on model perplexity/accuracy
 * (needs models and datasets that are not available) -- "parity unpinned" for that.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------ formats */

static const double E2M1_MAG[8] = {0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0};

/* value of a 4-bit E2M1 code: bit 3 = sign, bits 0..2 index the magnitudes above */
double oracle_e2m1_value(int code)
{
    double m = E2M1_MAG[code & 7];
    return (code & 8) ? -m : m;
}

/* value of an 8-bit E4M3 ("FN": finite + NaN, no infinities) code.
 * E = 0: (M/8) * 2^-6; E = 1..15: (1 + M/8) * 2^(E-7); 0x7F and 0xFF are NaN. */
double oracle_e4m3_value(int code)
{
    int s = (code >> 7) & 1, e = (code >> 3) & 15, m = code & 7;
    double v;
    if (e == 15 && m == 7) return NAN;
    if (e == 0) v = ldexp((double)m / 8.0, -6);
    else        v = ldexp(1.0 + (double)m / 8.0, e - 7);
    return s ? -v : v;
}

/* nearest magnitude code among codes 0..max_code whose values are val(code);
 * ties go to the even code; above the top value -> top code (saturation) */
static int nearest_code(double a, int max_code, const double *val)
{
    if (a >= val[max_code]) return max_code;      /* saturation */
    int best = 0;
    double bestd = fabs(a - val[0]);
    for (int c = 1; c <= max_code; ++c) {
        double d = fabs(a - val[c]);
        if (d < bestd || (d == bestd && (c & 1) == 0 && (best & 1) == 1)) {
            best = c; bestd = d;
        }
    }
    return best;
}

/* the 127 non-negative finite E4M3 magnitudes, tabulated once from the closed form */
static double E4M3_MAG[127];
static int e4m3_mag_ready = 0;
static void init_tables(void)
{
    if (e4m3_mag_ready) return;
    for (int c = 0; c <= 0x7E; ++c) E4M3_MAG[c] = oracle_e4m3_value(c);
    e4m3_mag_ready = 1;
}

int oracle_e2m1_encode(float x)
{
    int sign = signbit(x) ? 8 : 0;
    return sign | nearest_code(fabs((double)x), 7, E2M1_MAG);
}

int oracle_e4m3_encode(float x)
{
    int sign = signbit(x) ? 0x80 : 0;
    init_tables();
    return sign | nearest_code(fabs((double)x), 0x7E, E4M3_MAG);
}

static float bf16_to_float(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16; float f; memcpy(&f, &u, 4); return f;
}

/* ------------------------------------------------------ block-level pieces */

enum { BS = 16 };

/* dynamic-max scale code of a block (Section 3.3: activations; weights without clipping) */
static int block_dynamic_scale(const float *v, float s4)
{
    float amax = 0.0f;
    for (int i = 0; i < BS; ++i) { float a = fabsf(v[i]); if (a > amax) amax = a; }
    float k6 = 1.0f / (6.0f * s4);
    return oracle_e4m3_encode(amax * k6) & 0x7F;
}

/* NVFP4 encode of a block under scale code c; returns dequantized values too */
static void block_nvfp4(const float *v, int c, float s4, int *codes, float *dq)
{
    float d = (float)oracle_e4m3_value(c) * s4;
    if (d == 0.0f) {
        for (int i = 0; i < BS; ++i) { codes[i] = signbit(v[i]) ? 8 : 0; dq[i] = (float)oracle_e2m1_value(codes[i]) * d; }
        return;
    }
    float inv = 1.0f / d;
    for (int i = 0; i < BS; ++i) {
        codes[i] = oracle_e2m1_encode(v[i] * inv);
        dq[i] = (float)oracle_e2m1_value(codes[i]) * d;
    }
}

static void block_fp8(const float *v, float s8, int *codes, float *dq)
{
    float inv8 = 1.0f / s8;
    for (int i = 0; i < BS; ++i) {
        codes[i] = oracle_e4m3_encode(v[i] * inv8);
        dq[i] = (float)oracle_e4m3_value(codes[i]) * s8;
    }
}

/* Eq. 6 (mode 0) or Eq. 8 (mode 1), sequential fp32 sum */
static float block_score(const float *v, const float *f, const float *dq4, const float *dq8, int mode)
{
    float s = 0.0f;
    for (int i = 0; i < BS; ++i) {
        float e = (mode == 0) ? (v[i] - dq4[i]) : (dq4[i] - dq8[i]);
        float t = f[i] * e;
        t = t * e;
        s = s + t;
    }
    return s;
}

/* Eq. 11 objective for scale code c */
static float clip_objective(const float *v, const float *f, int c, float s4)
{
    int codes[BS]; float dq[BS];
    block_nvfp4(v, c, s4, codes, dq);
    float s = 0.0f;
    for (int i = 0; i < BS; ++i) {
        float e = dq[i] - v[i];
        float t = f[i] * e;
        t = t * e;
        s = s + t;
    }
    return s;
}

/* Eq. 11: brute force over the 126 positive finite E4M3 scale codes; the dynamic-max
 * code is the incumbent, a candidate replaces it only on strict improvement, codes
 * are visited in ascending order. */
int oracle_clip_search(const float *v, const float *f, float s4)
{
    int best = block_dynamic_scale(v, s4);
    float bestj = clip_objective(v, f, best, s4);
    for (int c = 1; c <= 0x7E; ++c) {
        float j = clip_objective(v, f, c, s4);
        if (j < bestj) { best = c; bestj = j; }
    }
    return best;
}

float oracle_clip_objective(const float *v, const float *f, int c, float s4)
{
    return clip_objective(v, f, c, s4);
}

static void write_block(int fp8, const int *c4, const int *c8, int sc,
                        uint8_t *codes4, uint8_t *codes8, uint8_t *scales, uint32_t *mask,
                        int64_t row, int64_t kb, int64_t K, int64_t mask_words)
{
    uint8_t *p4 = codes4 + (row * K + kb * BS) / 2;
    uint8_t *p8 = codes8 + row * K + kb * BS;
    if (fp8) {
        for (int i = 0; i < BS / 2; ++i) p4[i] = 0;
        for (int i = 0; i < BS; ++i) p8[i] = (uint8_t)c8[i];
        scales[row * (K / BS) + kb] = 0;
        mask[row * mask_words + kb / 32] |= (uint32_t)1 << (kb % 32);
    } else {
        for (int i = 0; i < BS / 2; ++i) p4[i] = (uint8_t)(c4[2 * i] | (c4[2 * i + 1] << 4));
        for (int i = 0; i < BS; ++i) p8[i] = 0;
        scales[row * (K / BS) + kb] = (uint8_t)sc;
    }
}

/* ------------------------------------------------------------ activations */

/* Online activation quantizer (Section 4.2).  X is bf16 [M, ldx]; fisher is per
 * input channel [K]; outputs are the canonical arrays:
 *   codes4 [M*K/2]  two E2M1 per byte, even element in the low nibble, 0 for FP8 blocks
 *   codes8 [M*K]    E4M3, 0 for FP4 blocks
 *   scales [M*K/16] E4M3 microscale, 0 for FP8 blocks
 *   mask   [M*ceil(K/16/32)] bit j of word w = block 32w+j, 1 = FP8
 *   scores [M*K/16] fp32 block scores
 * A block is FP8 iff score > tau (strict). */
void oracle_quantize_activations(const uint16_t *X, int64_t ldx, const float *fisher,
                                 int64_t M, int64_t K, float s4, int ratio, float s8_given, int mode, float tau,
                                 uint8_t *codes4, uint8_t *codes8, uint8_t *scales,
                                 uint32_t *mask, float *scores)
{
    int64_t KB = K / BS, MW = (KB + 31) / 32;
    float s8 = s8_given > 0.0f ? s8_given : ldexpf(s4, ratio);
    init_tables();
    memset(mask, 0, (size_t)(M * MW) * 4);
    #pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        for (int64_t kb = 0; kb < KB; ++kb) {
            float v[BS], dq4[BS], dq8[BS]; int c4[BS], c8[BS];
            for (int i = 0; i < BS; ++i) v[i] = bf16_to_float(X[m * ldx + kb * BS + i]);
            int sc = block_dynamic_scale(v, s4);
            block_nvfp4(v, sc, s4, c4, dq4);
            block_fp8(v, s8, c8, dq8);
            float score = block_score(v, fisher + kb * BS, dq4, dq8, mode);
            scores[m * KB + kb] = score;
            write_block(score > tau, c4, c8, sc, codes4, codes8, scales, mask, m, kb, K, MW);
        }
    }
}

/* ----------------------------------------------------------------- weights */

typedef struct { float score; int64_t idx; } scored_t;

static int cmp_scored(const void *a, const void *b)
{
    const scored_t *x = (const scored_t *)a, *y = (const scored_t *)b;
    if (x->score > y->score) return -1;
    if (x->score < y->score) return 1;
    return (x->idx < y->idx) ? -1 : (x->idx > y->idx);
}

/* Offline weight packer.  W bf16 [N, ldw], per-element Fisher [N, ldf].
 * s4_in = 0 -> derive the NVFP4 tensor scale as amax(W) / (6 * 448).
 * clip = 1 -> Eq. 11 search, else dynamic max.  The block score is taken under the
 * chosen scale.  fp8_fraction >= 0 -> exactly floor(R*B + 0.5) blocks with the
 * largest scores become FP8 (ties: lower linear block index first), tau_eff = the
 * smallest selected score; fp8_fraction < 0 -> FP8 iff score > tau.
 * Returns the tensor scale used. */
float oracle_quantize_weights(const uint16_t *W, int64_t ldw, const float *fisher, int64_t ldf,
                              int64_t N, int64_t K, float s4_in, int ratio, float s8_given, int mode, int clip,
                              double fp8_fraction, float tau,
                              uint8_t *codes4, uint8_t *codes8, uint8_t *scales,
                              uint32_t *mask, float *scores, float *tau_eff)
{
    int64_t KB = K / BS, MW = (KB + 31) / 32, B = N * KB;
    float s4 = s4_in;
    init_tables();
    if (s4 == 0.0f) {
        float amax = 0.0f;
        for (int64_t n = 0; n < N; ++n)
            for (int64_t k = 0; k < K; ++k) {
                float a = fabsf(bf16_to_float(W[n * ldw + k]));
                if (a > amax) amax = a;
            }
        s4 = amax / 2688.0f;
    }
    float s8 = s8_given > 0.0f ? s8_given : ldexpf(s4, ratio);
    uint8_t *sc_all = (uint8_t *)malloc((size_t)B);
    memset(mask, 0, (size_t)(N * MW) * 4);

    #pragma omp parallel for schedule(dynamic, 1)
    for (int64_t n = 0; n < N; ++n) {
        for (int64_t kb = 0; kb < KB; ++kb) {
            float v[BS], dq4[BS], dq8[BS]; int c4[BS], c8[BS];
            const float *f = fisher + n * ldf + kb * BS;
            for (int i = 0; i < BS; ++i) v[i] = bf16_to_float(W[n * ldw + kb * BS + i]);
            int sc = clip ? oracle_clip_search(v, f, s4) : block_dynamic_scale(v, s4);
            block_nvfp4(v, sc, s4, c4, dq4);
            block_fp8(v, s8, c8, dq8);
            scores[n * KB + kb] = block_score(v, f, dq4, dq8, mode);
            sc_all[n * KB + kb] = (uint8_t)sc;
        }
    }

    uint8_t *is8 = (uint8_t *)calloc((size_t)B, 1);
    float teff = tau;
    if (fp8_fraction >= 0.0) {
        int64_t k = (int64_t)floor(fp8_fraction * (double)B + 0.5);
        if (k > B) k = B;
        scored_t *s = (scored_t *)malloc((size_t)B * sizeof(scored_t));
        for (int64_t b = 0; b < B; ++b) { s[b].score = scores[b]; s[b].idx = b; }
        qsort(s, (size_t)B, sizeof(scored_t), cmp_scored);
        for (int64_t j = 0; j < k; ++j) is8[s[j].idx] = 1;
        teff = (k > 0) ? s[k - 1].score : INFINITY;
        free(s);
    } else {
        for (int64_t b = 0; b < B; ++b) is8[b] = scores[b] > tau;
    }
    if (tau_eff) *tau_eff = teff;

    for (int64_t n = 0; n < N; ++n) {
        for (int64_t kb = 0; kb < KB; ++kb) {
            float v[BS], dq4[BS], dq8[BS]; int c4[BS], c8[BS];
            for (int i = 0; i < BS; ++i) v[i] = bf16_to_float(W[n * ldw + kb * BS + i]);
            int sc = sc_all[n * KB + kb];
            block_nvfp4(v, sc, s4, c4, dq4);
            block_fp8(v, s8, c8, dq8);
            write_block(is8[n * KB + kb], c4, c8, sc, codes4, codes8, scales, mask, n, kb, K, MW);
        }
    }
    free(is8); free(sc_all);
    return s4;
}

/* -------------------------------------------------------------------- GEMM */

/* exact fp64 value of element k of a row given the canonical arrays */
static double decode_elem(const uint8_t *codes4, const uint8_t *codes8, const uint8_t *scales,
                          const uint32_t *mask, int64_t row, int64_t k, int64_t K,
                          double s4, double s8)
{
    int64_t KB = K / BS, MW = (KB + 31) / 32, kb = k / BS;
    int fp8 = (mask[row * MW + kb / 32] >> (kb % 32)) & 1;
    if (fp8) return oracle_e4m3_value(codes8[row * K + k]) * s8;
    uint8_t byte = codes4[(row * K + k) / 2];
    int code = (k & 1) ? (byte >> 4) : (byte & 15);
    return oracle_e2m1_value(code) * oracle_e4m3_value(scales[row * KB + kb]) * s4;
}

void oracle_decode(const uint8_t *codes4, const uint8_t *codes8, const uint8_t *scales,
                   const uint32_t *mask, int64_t rows, int64_t K, float s4, int ratio, float s8_given, double *out)
{
    double s8 = s8_given > 0.0f ? (double)s8_given : ldexp((double)s4, ratio);
    #pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t k = 0; k < K; ++k)
            out[r * K + k] = decode_elem(codes4, codes8, scales, mask, r, k, K, (double)s4, s8);
}

/* Y[m,n] = sum_k A[m,k] W[n,k] in fp64 over decoded operands (Section 3: Y = W x X;
 * Section 4.1: per block pair the product of the two formats, accumulated).  S holds
 * sum_k |A||W|, the normaliser of the error bound.  A and Wt are decoded [rows, K]. */
void oracle_linear(const double *A, const double *Wd, int64_t M, int64_t N, int64_t K,
                   double *Y, double *S)
{
    #pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < N; ++n) {
            double y = 0.0, s = 0.0;
            for (int64_t k = 0; k < K; ++k) {
                double p = A[m * K + k] * Wd[n * K + k];
                y += p; s += fabs(p);
            }
            Y[m * N + n] = y;
            if (S) S[m * N + n] = s;
        }
}

/* the same sum for a list of output coordinates, decoding on the fly (full-size
 * configurations, sampled outputs) */
void oracle_linear_sampled(const uint8_t *a4, const uint8_t *a8, const uint8_t *asc, const uint32_t *am,
                           float a_s4, int a_ratio, float a_s8_given,
                           const uint8_t *w4, const uint8_t *w8, const uint8_t *wsc, const uint32_t *wm,
                           float w_s4, int w_ratio, float w_s8_given, int64_t K,
                           int64_t nsamp, const int64_t *ms, const int64_t *ns, double *Y, double *S)
{
    double as8 = a_s8_given > 0.0f ? (double)a_s8_given : ldexp((double)a_s4, a_ratio);
    double ws8 = w_s8_given > 0.0f ? (double)w_s8_given : ldexp((double)w_s4, w_ratio);
    #pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < nsamp; ++j) {
        double y = 0.0, s = 0.0;
        for (int64_t k = 0; k < K; ++k) {
            double a = decode_elem(a4, a8, asc, am, ms[j], k, K, (double)a_s4, as8);
            double w = decode_elem(w4, w8, wsc, wm, ns[j], k, K, (double)w_s4, ws8);
            y += a * w; s += fabs(a * w);
        }
        Y[j] = y; S[j] = s;
    }
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
