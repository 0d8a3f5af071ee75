/*
 * mxq_oracle.c -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, single-precision CPU statement of block-wise microscaled FP4 (E2M1)
 * quantization with per-block scale selection and MSE scoring, written from the paper
 * "Finer is Better (with the Right Scaling)".  It exists so that the CUDA library can be
 * checked against something that a reader can compare with the paper by eye.  Only the
 * tests, the smoke check and the benchmark's cpu-baseline leg may call it.  It shares no
 * code, header, table or constant generator with the CUDA library.
 *
 * Build:  gcc -O2 -std=c11 -ffp-contract=off -fno-fast-math -fPIC -shared -pthread
 * (-ffp-contract=off: every float operation below is ONE IEEE-754 binary32
 *  round-to-nearest-even operation; fmaf() is the only fused operation and it is explicit.)
 *
 * Precision.  The method's outputs are integers (FP4 codes, scale bytes) decided by floating
 * point, so both sides must decide in the same precision: binary32, operations in the order
 * written here.  Tensor MSE is accumulated in binary64.
 *
 * Pins (tests/test_oracle_*.py): exhaustive format tables against the values the paper prints
 * (E2M1 value set, eps = 2^-9 for E4M3, M_max = 6) and against ml_dtypes bit patterns; scale and
 * element rounding against exact rational arithmetic; Eq. 1 on hand-worked blocks; per-block
 * orderings brute <= 4-over-6 <= abs-max and prevent-zero <= plain; exact reconstruction of
 * on-grid blocks; finer-is-better for the brute-force optimum; sign and power-of-two symmetries.
 * UE5M3: the paper names the format but does not define bias, maximum or NaN code; the table
 * below is a stated reading, so the UE5M3 *format definition* is "parity unpinned" by the paper
 * (its rounding and everything built on it is pinned like the other formats).
 */
#include <math.h>
#include <pthread.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

enum { ORC_F32 = 0, ORC_BF16 = 1 };
enum { ORC_UE8M0 = 0, ORC_UE4M3 = 1, ORC_UE5M3 = 2 };
enum { ORC_ABSMAX = 0, ORC_ABSMAX_PZ = 1, ORC_4O6 = 2, ORC_4O6_PZ = 3, ORC_BRUTE = 4, ORC_BRUTE_PZ = 5, ORC_ABSMAX_OCP = 6,
       ORC_ABSMAX_CLIP7 = 7 };

/* ---------------------------------------------------------------------------------------------
 * Number formats (Background; Experimental Setup).
 * ------------------------------------------------------------------------------------------- */

/* FP4 E2M1 magnitudes, Experimental Setup: +-{0, 0.5, 1, 1.5, 2, 3, 4, 6}.  A 4-bit code is
 * sign<<3 | index into this list (OCP E2M1 bit order s.ee.m equals value order). */
static const float E2M1_GRID[8] = {0.0f, 0.5f, 1.0f, 1.5f, 2.0f, 3.0f, 4.0f, 6.0f};

/* Number of finite, usable codes of a block-scale format: codes 0 .. count-1. */
int mxq_oracle_num_codes(int fmt)
{
    switch (fmt) {
    case ORC_UE8M0: return 255; /* 0xFF reserved (NaN) */
    case ORC_UE4M3: return 127; /* sign bit unused; 0x7F is NaN in OFP8 E4M3 */
    case ORC_UE5M3: return 255; /* reading: only 0xFF reserved */
    default: return 0;
    }
}

/* Decoded value of scale code `code`.
 * UE8M0: 2^(code-127).
 * UE4M3: exponent bias 7, 3 mantissa bits, subnormals m*2^-9; smallest nonzero 2^-9 as the paper
 *        states for E4M3 (Eq. 3 text); largest finite 448.
 * UE5M3: reading (paper silent): exponent bias 15, 3 mantissa bits, subnormals m*2^-17,
 *        largest finite 1.75*2^16. */
float mxq_oracle_scale_value(int fmt, int code)
{
    if (code < 0 || code >= mxq_oracle_num_codes(fmt)) return NAN;
    if (fmt == ORC_UE8M0) return ldexpf(1.0f, code - 127);
    int e = code >> 3, m = code & 7;
    int bias = (fmt == ORC_UE4M3) ? 7 : 15;
    if (e == 0) return ldexpf((float)m, 1 - bias - 3);
    return ldexpf(1.0f + (float)m / 8.0f, e - bias);
}

/* Round_SF of Eq. 2 for the 8-bit floating-point scale formats: round-to-nearest-even onto the
 * format's value lattice, clipped to the largest finite value.  Written as a search over the
 * table so that it can be checked by eye: find the two neighbouring codes, compare with their
 * midpoint (exact in double: both neighbours have <= 4 significant bits), ties to the even code. */
static int round_sf_nearest_even(int fmt, float w)
{
    int n = mxq_oracle_num_codes(fmt);
    if (!(w > 0.0f)) return 0;
    if (w >= mxq_oracle_scale_value(fmt, n - 1)) return n - 1;
    int lo = 0;
    for (int c = 1; c < n; ++c)
        if (mxq_oracle_scale_value(fmt, c) <= w) lo = c;
    int hi = lo + 1;
    double mid = ((double)mxq_oracle_scale_value(fmt, lo) + (double)mxq_oracle_scale_value(fmt, hi)) / 2.0;
    if ((double)w < mid) return lo;
    if ((double)w > mid) return hi;
    return (lo % 2 == 0) ? lo : hi;
}

/* Eq. 1 for the power-of-two format: S = 2^floor(log2 w) with w = amax / M_max, i.e. the largest
 * representable power of two that is <= w, clamped to the format's range. */
static int round_sf_pow2_floor(float w)
{
    int lo = 0;
    for (int c = 0; c < 255; ++c)
        if (ldexpf(1.0f, c - 127) <= w) lo = c;
    return lo;
}

/* Scale code chosen for the target w = amax / M (already divided).  UE8M0 follows Eq. 1 (floor),
 * the FP8 formats follow Eq. 2 (RNE + clip). */
int mxq_oracle_round_scale(int fmt, float w)
{
    if (fmt == ORC_UE8M0) return round_sf_pow2_floor(w);
    return round_sf_nearest_even(fmt, w);
}

/* quant(): round-to-nearest-even of |t| onto the E2M1 magnitudes with saturation at 6; returns
 * the magnitude index 0..7.  Midpoints 0.25 0.75 1.25 1.75 2.5 3.5 5 go to the even index. */
int mxq_oracle_e2m1_index(float t)
{
    float a = fabsf(t);
    if (a >= 6.0f) return 7;
    int lo = 0;
    for (int k = 1; k < 8; ++k)
        if (E2M1_GRID[k] <= a) lo = k;
    float mid = (E2M1_GRID[lo] + E2M1_GRID[lo + 1]) / 2.0f; /* exact */
    if (a < mid) return lo;
    if (a > mid) return lo + 1;
    return (lo % 2 == 0) ? lo : lo + 1;
}

float mxq_oracle_e2m1_value(int code4)
{
    float m = E2M1_GRID[code4 & 7];
    return (code4 & 8) ? -m : m;
}

static float widen_bf16(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

static uint16_t narrow_bf16_rne(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    return (uint16_t)(u >> 16);
}

static float load_elem(const void *x, int dtype, size_t i)
{
    return dtype == ORC_BF16 ? widen_bf16(((const uint16_t *)x)[i]) : ((const float *)x)[i];
}

/* ---------------------------------------------------------------------------------------------
 * One block, one scale code: quantize every element and score the block.
 *   D    = fl32(S * g)                      effective decode scale (S block scale, g tensor scale)
 *   t    = fl32(v / D)                      "v_i -> quant(v_i / S)"
 *   code = signbit(v) << 3 | RNE_E2M1(|t|)  (a zero scale sets every magnitude to zero)
 *   e    = fma(-grid(code), D, v);  sse = fma(e, e, sse), elements in order, sse starts at 0.
 * codes4 (may be NULL) receives one 4-bit code per element, unpacked.
 * ------------------------------------------------------------------------------------------- */
static float eval_block(const float *v, int B, int fmt, int code, float g, uint8_t *codes4)
{
    float S = mxq_oracle_scale_value(fmt, code);
    float D = S * g;
    float sse = 0.0f;
    for (int i = 0; i < B; ++i) {
        int idx = 0;
        if (D != 0.0f) {
            float t = v[i] / D;
            idx = mxq_oracle_e2m1_index(t);
        }
        int c4 = (signbit(v[i]) ? 8 : 0) | idx;
        if (codes4) codes4[i] = (uint8_t)c4;
        float q = mxq_oracle_e2m1_value(c4);
        float e = fmaf(-q, D, v[i]);
        sse = fmaf(e, e, sse);
    }
    return sse;
}

/* Exposed for the pins: SSE of one block under one given scale code. */
float mxq_oracle_block_sse(const float *v, int B, int fmt, int code, float g, uint8_t *codes4)
{
    return eval_block(v, B, fmt, code, g, codes4);
}

/* Eq. 2 candidate for divisor M (6 = standard abs-max, 4 = the second 4-over-6 candidate), with
 * the optional Eq. 3 clamp.  Hierarchical scaling: the block scale is chosen for inputs already
 * divided by the tensor scale, i.e. the target comes from amax / g. */
static int absmax_code(float amax, float g, float M, int fmt, int prevent_zero)
{
    float u = amax / g;
    float w = u / M;
    int c = mxq_oracle_round_scale(fmt, w);
    /* Eq. 3: S = max(S, eps_SF), eps_SF = smallest nonzero value of the format.  For the FP8
     * formats that is code 1; in UE8M0 every code is nonzero, so the clamp changes nothing. */
    if (prevent_zero && fmt != ORC_UE8M0 && c < 1) c = 1;
    return c;
}

/* The power-of-two rule as the OCP MX specification words it (Background: the paper paraphrases
 * it in prose and prints Eq. 1, which differs): the shared exponent is the exponent of the block
 * maximum minus the exponent of the largest element value, S = 2^(floor(log2 amax) - 2) for E2M1
 * (6 = 1.5 * 2^2).  The maximum then lands in [4, 8) and is clipped when it exceeds 6.  UE8M0
 * only; amax is first adjusted by the tensor scale like in the other recipes. */
int mxq_oracle_ocp_code(float amax, float g)
{
    float u = amax / g;
    if (!(u > 0.0f)) return 0;
    if (isinf(u)) return 254;     /* amax / g overflowed: the largest scale, as the floor rule of Eq. 1 gives */
    int e;
    (void)frexpf(u, &e);          /* u = f * 2^e, 0.5 <= f < 1: floor(log2 u) = e - 1 */
    int c = 127 + (e - 1) - 2;
    if (c < 0) c = 0;
    if (c > 254) c = 254;
    return c;
}

/* The power-of-two scale that maps the block maximum into [3.5, 7) (Background: the clipping
 * recipe of a cited work; a maximum that lands above 6 is clipped): the largest e with
 * 3.5 * 2^e <= amax / g, written out as that search.  UE8M0 only. */
int mxq_oracle_clip7_code(float amax, float g)
{
    float u = amax / g;
    if (!(u > 0.0f)) return 0;
    if (isinf(u)) return 254;
    int e;
    (void)frexpf(u, &e);                              /* u = f * 2^e with f < 1, so 3.5 * 2^e > u: start above */
    while ((double)ldexp(3.5, e) > (double)u) --e;    /* 3.5 * 2^e is exact in binary64 */
    int c = 127 + e;
    if (c < 0) c = 0;
    if (c > 254) c = 254;
    return c;
}

/* Choose the scale code of one block by recipe; returns the code, writes the block's SSE. */
static int choose_code(const float *v, int B, int fmt, int recipe, float g, float *sse_out)
{
    float amax = 0.0f;
    for (int i = 0; i < B; ++i)
        if (fabsf(v[i]) > amax) amax = fabsf(v[i]);

    int pz = (recipe == ORC_ABSMAX_PZ || recipe == ORC_4O6_PZ || recipe == ORC_BRUTE_PZ);
    int best;
    float best_sse;

    if (recipe == ORC_ABSMAX || recipe == ORC_ABSMAX_PZ) {
        best = absmax_code(amax, g, 6.0f, fmt, pz);
        best_sse = eval_block(v, B, fmt, best, g, NULL);
    } else if (recipe == ORC_ABSMAX_OCP || recipe == ORC_ABSMAX_CLIP7) {
        best = (recipe == ORC_ABSMAX_OCP) ? mxq_oracle_ocp_code(amax, g) : mxq_oracle_clip7_code(amax, g);
        best_sse = eval_block(v, B, fmt, best, g, NULL);
    } else if (recipe == ORC_4O6 || recipe == ORC_4O6_PZ) {
        /* Eq. 4: argmin over M in {4, 6} of the block error; a tie keeps M = 6. */
        int c6 = absmax_code(amax, g, 6.0f, fmt, pz);
        int c4 = absmax_code(amax, g, 4.0f, fmt, pz);
        float s6 = eval_block(v, B, fmt, c6, g, NULL);
        float s4 = eval_block(v, B, fmt, c4, g, NULL);
        if (s4 < s6) { best = c4; best_sse = s4; } else { best = c6; best_sse = s6; }
    } else {
        /* Brute force: every finite code of the format (prevent-zero: every code whose value is
         * nonzero); smallest SSE wins, equal SSE keeps the smaller code.  A code whose decode
         * scale S*g is not a finite float cannot be used and is skipped. */
        int n = mxq_oracle_num_codes(fmt);
        int first = (pz && fmt != ORC_UE8M0) ? 1 : 0;
        best = -1;
        best_sse = 0.0f;
        for (int c = first; c < n; ++c) {
            float D = mxq_oracle_scale_value(fmt, c) * g;
            if (!isfinite(D)) continue;
            float s = eval_block(v, B, fmt, c, g, NULL);
            if (best < 0 || s < best_sse) { best = c; best_sse = s; }
        }
        if (best < 0) { best = first; best_sse = eval_block(v, B, fmt, best, g, NULL); }
    }
    *sse_out = best_sse;
    return best;
}

/* ---------------------------------------------------------------------------------------------
 * Whole tensors.
 * ------------------------------------------------------------------------------------------- */
static void quantize_range(const void *x, int dtype, size_t b0, size_t b1, int B, int fmt, int recipe, float g,
                           uint8_t *codes, uint8_t *scales, float *block_sse)
{
    float v[64];
    uint8_t c4[64];
    for (size_t b = b0; b < b1; ++b) {
        for (int i = 0; i < B; ++i) v[i] = load_elem(x, dtype, b * (size_t)B + (size_t)i);
        float sse;
        int code = choose_code(v, B, fmt, recipe, g, &sse);
        float sse2 = eval_block(v, B, fmt, code, g, c4);
        (void)sse2; /* same function of (block, code): identical to sse */
        if (scales) scales[b] = (uint8_t)code;
        if (block_sse) block_sse[b] = sse;
        if (codes) /* element 2j in the low nibble, 2j+1 in the high nibble */
            for (int i = 0; i < B; i += 2) codes[(b * (size_t)B + (size_t)i) / 2] = (uint8_t)(c4[i] | (c4[i + 1] << 4));
    }
}

/* x: n elements (float or bf16 bit patterns), n a multiple of B, B in {2,4,8,16,32,64}.
 * codes: n/2 bytes; scales: n/B bytes; block_sse: n/B floats (each may be NULL).
 * Returns 0, or -1 on a bad argument. */
int mxq_oracle_quantize(const void *x, int dtype, size_t n, int B, int fmt, int recipe, float g, uint8_t *codes,
                        uint8_t *scales, float *block_sse)
{
    if (!x || n == 0 || B < 2 || B > 64 || (B & (B - 1)) || n % (size_t)B) return -1;
    if (mxq_oracle_num_codes(fmt) == 0 || recipe < 0 || recipe > ORC_ABSMAX_CLIP7) return -1;
    if ((recipe == ORC_ABSMAX_OCP || recipe == ORC_ABSMAX_CLIP7) && fmt != ORC_UE8M0) return -1;
    if (!(g > 0.0f) || !isfinite(g)) return -1;
    quantize_range(x, dtype, 0, n / (size_t)B, B, fmt, recipe, g, codes, scales, block_sse);
    return 0;
}

struct mt_job {
    const void *x; int dtype; size_t b0, b1; int B, fmt, recipe; float g;
    uint8_t *codes, *scales; float *sse;
};

static void *mt_entry(void *p)
{
    struct mt_job *j = (struct mt_job *)p;
    quantize_range(j->x, j->dtype, j->b0, j->b1, j->B, j->fmt, j->recipe, j->g, j->codes, j->scales, j->sse);
    return NULL;
}

/* Same result as mxq_oracle_quantize; blocks are independent, so they are split evenly over
 * `threads` host threads (used only to report a host-cores baseline). */
int mxq_oracle_quantize_mt(const void *x, int dtype, size_t n, int B, int fmt, int recipe, float g, uint8_t *codes,
                           uint8_t *scales, float *block_sse, int threads)
{
    if (threads <= 1) return mxq_oracle_quantize(x, dtype, n, B, fmt, recipe, g, codes, scales, block_sse);
    if (!x || n == 0 || B < 2 || B > 64 || (B & (B - 1)) || n % (size_t)B) return -1;
    if (mxq_oracle_num_codes(fmt) == 0 || recipe < 0 || recipe > ORC_ABSMAX_CLIP7) return -1;
    if ((recipe == ORC_ABSMAX_OCP || recipe == ORC_ABSMAX_CLIP7) && fmt != ORC_UE8M0) return -1;
    if (!(g > 0.0f) || !isfinite(g)) return -1;
    if (threads > 256) threads = 256;
    pthread_t tid[256];
    struct mt_job job[256];
    size_t nb = n / (size_t)B;
    for (int t = 0; t < threads; ++t) {
        struct mt_job j = {x, dtype, nb * (size_t)t / (size_t)threads, nb * (size_t)(t + 1) / (size_t)threads,
                           B, fmt, recipe, g, codes, scales, block_sse};
        job[t] = j;
        pthread_create(&tid[t], NULL, mt_entry, &job[t]);
    }
    for (int t = 0; t < threads; ++t) pthread_join(tid[t], NULL);
    return 0;
}

/* Per-tensor abs-max (first stage of hierarchical scaling). */
float mxq_oracle_tensor_amax(const void *x, int dtype, size_t n)
{
    float amax = 0.0f;
    for (size_t i = 0; i < n; ++i) {
        float a = fabsf(load_elem(x, dtype, i));
        if (a > amax) amax = a;
    }
    return amax;
}

/* Tensor MSE = (sum over blocks of the block SSE) / n, summed in block order in binary64. */
double mxq_oracle_tensor_mse(const float *block_sse, size_t n_blocks, size_t n)
{
    double s = 0.0;
    for (size_t b = 0; b < n_blocks; ++b) s += (double)block_sse[b];
    return s / (double)n;
}

/* De-quantization is a multiplication by the scale: x_hat = fl32(grid(code) * D), D = fl32(S * g).
 * out_dtype ORC_BF16 additionally rounds x_hat to bf16 (RNE). */
int mxq_oracle_dequantize(const uint8_t *codes, const uint8_t *scales, size_t n, int B, int fmt, float g, void *out,
                          int out_dtype)
{
    if (!codes || !scales || !out || n == 0 || n % (size_t)B) return -1;
    for (size_t i = 0; i < n; ++i) {
        int sc = scales[i / (size_t)B];
        if (sc >= mxq_oracle_num_codes(fmt)) return -1;
        float D = mxq_oracle_scale_value(fmt, sc) * g;
        int c4 = (codes[i / 2] >> ((i & 1) ? 4 : 0)) & 15;
        float xh = mxq_oracle_e2m1_value(c4) * D;
        if (out_dtype == ORC_BF16) ((uint16_t *)out)[i] = narrow_bf16_rne(xh);
        else ((float *)out)[i] = xh;
    }
    return 0;
}

/* ---------------------------------------------------------------------------------------------
 * Analysis outputs of the numerical study and the appendix (Results, numerical study; Appendix:
 * "Clipping only MSE", entry and scale histograms).
 * ------------------------------------------------------------------------------------------- */

/* Clipping part of the block SSE: the error of the elements whose scaled magnitude exceeds the
 * largest FP4 value, |fl32(v / D)| > 6 (they are all mapped to +-6).  Same arithmetic and element
 * order as the block SSE, restricted to those elements; a zero scale clips nothing (its error is
 * underflow, not clipping).  scales: one code per block, as written by the quantizer. */
int mxq_oracle_block_clip_sse(const void *x, int dtype, size_t n, int B, int fmt, const uint8_t *scales, float g,
                              float *out_clip_sse)
{
    if (!x || !scales || !out_clip_sse || n == 0 || B < 2 || B > 64 || n % (size_t)B) return -1;
    for (size_t b = 0; b < n / (size_t)B; ++b) {
        if (scales[b] >= mxq_oracle_num_codes(fmt)) return -1;
        float D = mxq_oracle_scale_value(fmt, scales[b]) * g;
        float sse = 0.0f;
        for (int i = 0; i < B; ++i) {
            float v = load_elem(x, dtype, b * (size_t)B + (size_t)i);
            if (D == 0.0f) continue;
            float t = v / D;
            if (fabsf(t) > 6.0f) {
                float q = signbit(v) ? -6.0f : 6.0f;
                float e = fmaf(-q, D, v);
                sse = fmaf(e, e, sse);
            }
        }
        out_clip_sse[b] = sse;
    }
    return 0;
}

/* Histograms of the quantized entries (16 bins: the 4-bit code, sign included) and of the block
 * scale codes (256 bins).  Counts are ADDED to the arrays. */
int mxq_oracle_histograms(const uint8_t *codes, const uint8_t *scales, size_t n, int B, uint64_t *code_hist,
                          uint64_t *scale_hist)
{
    if (!codes || !scales || !code_hist || !scale_hist || n == 0 || n % (size_t)B) return -1;
    for (size_t i = 0; i < n; ++i) code_hist[(codes[i / 2] >> ((i & 1) ? 4 : 0)) & 15] += 1;
    for (size_t b = 0; b < n / (size_t)B; ++b) scale_hist[scales[b]] += 1;
    return 0;
}

/* MSE of consecutive segments of equal length (one sigma of the numerical study per segment):
 * out[s] = (sum of the block SSEs of segment s) / elems_per_segment, in binary64, block order. */
int mxq_oracle_segment_mse(const float *block_sse, size_t n_blocks, size_t blocks_per_segment, size_t elems_per_segment,
                           double *out)
{
    if (!block_sse || !out || blocks_per_segment == 0 || n_blocks % blocks_per_segment || elems_per_segment == 0) return -1;
    for (size_t s = 0; s < n_blocks / blocks_per_segment; ++s) {
        double acc = 0.0;
        for (size_t b = 0; b < blocks_per_segment; ++b) acc += (double)block_sse[s * blocks_per_segment + b];
        out[s] = acc / (double)elems_per_segment;
    }
    return 0;
}
