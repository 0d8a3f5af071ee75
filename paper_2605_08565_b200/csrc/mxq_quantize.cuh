// Fused one-pass quantization kernels: block amax -> scale code -> FP4 codes -> block SSE.
//   SINGLE  abs-max (Eq. 2; Eq. 1 for UE8M0), optional prevent-zero clamp (Eq. 3)
//   DUAL    4-over-6 (Eq. 4): candidates for M = 6 and M = 4, keep the smaller SSE
//
// Work layout.  One thread owns a chunk of consecutive elements (at least 64 bytes of input and
// at least one block) and walks it in groups of max(B, 8) elements (one block, or 8/B small
// blocks), so every per-block quantity lives in registers and the SSE is accumulated in element
// order.  Blocks of 32 and 64 elements are walked in parts of 16 (quantize_long_block()).  CTAs
// are persistent (grid = SMs x resident CTAs) and build the per-code table once.
//
// Input staging, chunks of 64 bytes.  Every thread copies ITS OWN next chunk into ITS OWN column
// of a two-slot shared-memory ring with asynchronous 16-byte copies (cp.async.ca: the 128-byte
// line that the first piece brings into L1 also serves the thread's other pieces and its
// neighbour) and waits for it with cp.async.wait_group.  The data never crosses threads, so no
// barrier of any kind is involved and nothing can wait forever.  One chunk per thread is in
// flight while the current one is processed, independent of how many registers the arithmetic
// needs; a third slot was measured and loses (the extra shared memory leaves too little L1 for
// fp32 input).  Slot layout: piece k of thread t sits at ((slot * PIECES + k) * 256 + t) * 16, so
// both the asynchronous writes and the later 128-bit reads of a warp are contiguous (no bank
// conflict).  Chunks above 64 bytes are copied by the warp together (stage_warp_chunks()) and
// handed over with a __syncwarp().
//
// Arithmetic per element (kernel time follows the number of warp instructions): bf16 -> binary32
// by a mixed-precision add of -0 (FMA pipe); the exact quotient by the decode scale, two elements
// per instruction (reciprocal multiply + one residual correction; for bf16 input and decode scales
// of at most four significant bits, or long ones whose reciprocal passed the per-launch check, a single
// multiply rounded toward zero); half an FP4 pack, half an FP4
// unpack; the residual as fma.rn.f32.f16 straight from the unpacked f16 grid value whenever the
// decode scales of the group are exactly representable in f16 (always, for UE4M3 without a tensor
// scale), else an f16->f32 convert plus an FFMA; the square-accumulate FMA, for 4-over-6 one
// fma.rn.f32x2 serving both candidates.  Blocks whose numbers fall outside the ranges these
// shortcuts need are redone with IEEE divisions (general path).
//
// Variants of the chunk loop inside one kernel, chosen once per launch after the table is built: the
// lean loop (see quantize_chunk) when no block can leave the shortcuts, the general loop otherwise.
// Every thread also adds the SSEs of its blocks in binary64; a launch that was given a partial-sum
// array (mxq_quantize_mse) ends with a fixed-order sum over the CTA.  The BATCH instantiation walks a
// list of tensors in one launch (quantize_batch_body()).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <atomic>
#include <type_traits>

#include "mxq_device.cuh"
#include "mxq_internal.h"

namespace mxq {

// Per-code table entry, one 128-bit shared-memory read per block and candidate:
//   x  D = fl32(value(c) * g); NaN for codes that do not exist
//   y  R = RN(1 / D) when 2^-60 <= D <= 2^60, else 0
//   z  bits: f16(-D) in the low half; in a bf16 kernel under a tensor scale that is not a power of two,
//      the reciprocal for the one-multiply quotient instead (R or a neighbour of it, see
//      build_quant_tables())
//   w  0: general path only; 1: shortcuts valid; 2: shortcuts valid and -D exact in f16; 3: as 2,
//      and D has at most four significant bits (every decode scale of the FP8 and power-of-two
//      formats when the tensor scale is a power of two).  Where z holds a reciprocal, w is 0 or 1.
//      D = 0 counts as valid with R = 0: every quotient comes out as a zero with the sign of v.
struct QuantTables {
    float4 E[256];
};

// Does the FP4 code of RZ(v * R) equal the FP4 code of fl32(v / D) for EVERY bf16 value v?  (D a
// normal binary32 number, R within a few units in the last place of 1 / D.)  Both codes are
// non-decreasing step functions of v >= 0 (and odd in v), so they agree everywhere iff they agree where
// either of them steps.  The steps are next to the seven points M * D, M a rounding midpoint of the FP4
// grid: the product and the true quotient differ by less than 2^-21 relative, bf16 values are at least
// 2^-8 apart, so at the second bf16 value above M * D both are safely above M and at the first one
// below floor_bf16(M * D) both safely below.  That leaves v0 = floor_bf16(M * D) and the bf16 value
// after it: two values per midpoint, tried here with the very instructions the hot loop uses (this
// function does one midpoint).
__device__ __forceinline__ bool one_multiply_codes_agree_at(float D, float R, float M) {
    const uint32_t b0 = __float_as_uint(__fmul_rz(M, D)) & 0xFFFF0000u;   // floor to 8 significant bits
    const float v0 = __uint_as_float(b0), v1 = __uint_as_float(b0 + 0x10000u);
    uint32_t codes;   // byte 0: {fl(v0 / D), RZ(v0 R)}, byte 1: the same for v1, FP4 codes in the two nibbles
    asm("{\n"
        " .reg .b8 b0, b1;\n"
        " cvt.rn.satfinite.e2m1x2.f32 b0, %1, %2;\n"
        " cvt.rn.satfinite.e2m1x2.f32 b1, %3, %4;\n"
        " mov.b32 %0, {b0, b1, b0, b1};\n"
        "}"
        : "=r"(codes)
        : "f"(__fdiv_rn(v0, D)), "f"(__fmul_rz(v0, R)), "f"(__fdiv_rn(v1, D)), "f"(__fmul_rz(v1, R)));
    return (((codes >> 4) ^ codes) & 0x0F0Fu) == 0u;
}

// Builds the table.  first_bad: the smallest code of the format whose class is below 3, or
// num_codes(FMT) if every code has class 3.  Returns (CTA-uniform) whether the one-multiply quotient
// with the reciprocals in E[].z may be used for every entry of class 1 (BF16_IN kernels under a tensor
// scale that is not a power of two; false otherwise).
//
// The one-multiply quotient under such a tensor scale.  Decode scales then have 24 significant bits, and
// whether RZ(v * R) has the FP4 code of fl(v / D) for every bf16 v depends on how the roundings fall
// where a bf16 value lies within 2^-23 or so of M * D.  With g = amax / 2688 from a bf16 amax that
// happens for most significands (v / D is then a ratio of small integers and hits midpoints exactly in
// real arithmetic; RN(1 / D) alone passes for 40 of the 128 amax significands).  It depends on the
// significand of D only (v, D and the quotient all scale by powers of two), and the scales of a table
// have at most eight significands: those of fl((1 + m / 8) * g).  So the check runs per significand
// class, for three candidate reciprocals (RN(1 / D), the float above it, the float below it) and the
// seven midpoints, on 168 threads, with the tensor scale's significand moved to [1, 2).  Each class
// takes the first candidate that passes at all seven midpoints (126 of those 128 significands then
// pass in every class); an entry records it only if its own significand bits are those of its class
// (always, unless g is denormal).  If some class has no passing candidate the launch keeps the
// corrected quotient throughout.
template <int FMT, bool BF16_IN>
__device__ __forceinline__ bool build_quant_tables(QuantTables& T, float g, int& first_bad) {
    static_assert(kThreads == 256, "one thread per table entry");
    __shared__ int leading_good[kThreads / 32];   // per warp: how many of its 32 codes, from the first on, have class 3
    __shared__ uint32_t class_sig[8];             // significand bits of fl((1 + m / 8) * g)
    __shared__ __align__(8) uint8_t cand_ok[8][3][8];   // [m][candidate][j]: midpoint j agrees ([..][7] = 1)
    const int c = threadIdx.x;
    const bool check = BF16_IN && (__float_as_uint(g) & 0x007FFFFFu) != 0u;   // a power of two keeps every scale short
    if (check) {                                  // CTA-uniform
        if (c < 8 * 21) {
            const int m = c / 21, r = c - 21 * m, cand = r / 7, j = r - 7 * cand;
            const float gn = __uint_as_float((__float_as_uint(g) & 0x007FFFFFu) | 0x3F800000u);
            const float Dr = __fmul_rn(1.0f + 0.125f * (float)m, gn);
            const float Rc = __uint_as_float(__float_as_uint(__frcp_rn(Dr)) + (cand == 0 ? 0u : (cand == 1 ? 1u : 0xFFFFFFFFu)));
            const float M = (j < 4) ? 0.25f + 0.5f * (float)j : (j == 4 ? 2.5f : (j == 5 ? 3.5f : 5.0f));
            cand_ok[m][cand][j] = one_multiply_codes_agree_at(Dr, Rc, M) ? 1 : 0;
            if (j == 0) cand_ok[m][cand][7] = 1;
            if (r == 0) class_sig[m] = __float_as_uint(Dr) & 0x007FFFFFu;
        }
        __syncthreads();
    }
    float D = __uint_as_float(0x7FC00000u), R = 0.0f, w = 0.0f;
    uint32_t z = 0;
    bool vote = true;
    if (c < num_codes(FMT)) {
        const float S = scale_value(FMT, c);
        D = __fmul_rn(S, g);
        const bool in_range = (D >= kFastMin && D <= kFastMax);
        if (in_range || D == 0.0f) {
            if (in_range) R = __frcp_rn(D);
            if (check) {
                w = 1.0f;
                if (in_range) {
                    const int m = (__float_as_uint(S) >> 20) & 7;
                    constexpr unsigned long long kAll = 0x0101010101010101ull;
                    const unsigned long long* ok = reinterpret_cast<const unsigned long long*>(cand_ok[m]);
                    const int cand = ok[0] == kAll ? 0 : (ok[1] == kAll ? 1 : (ok[2] == kAll ? 2 : 3));
                    vote = cand < 3 && (__float_as_uint(D) & 0x007FFFFFu) == class_sig[m];
                    z = __float_as_uint(R) + (cand == 1 ? 1u : (cand == 2 ? 0xFFFFFFFFu : 0u));
                }
            } else {
                const __half hD = __float2half_rn(-D);
                z = (uint32_t)__half_as_ushort(hD);
                w = (__half2float(hD) == -D) ? 2.0f : 1.0f;
                if (w == 2.0f && (__float_as_uint(D) & 0x000FFFFFu) == 0u) w = 3.0f;
            }
        }
    }
    T.E[c] = make_float4(D, R, __uint_as_float(z), w);
    const uint32_t good = __ballot_sync(0xFFFFFFFFu, w == 3.0f);
    if ((c & 31) == 0) leading_good[c >> 5] = (good == 0xFFFFFFFFu) ? 32 : (__ffs(~good) - 1);
    const bool all_voted = __syncthreads_and(vote) != 0;
    int fb = 0;
#pragma unroll
    for (int wp = 0; wp < kThreads / 32; ++wp) {
        if (fb == 32 * wp) fb += leading_good[wp];
    }
    first_bad = min(fb, num_codes(FMT));
    return check && all_voted;
}

// fl32(v / D) by a reciprocal multiply and ONE residual correction, R = RN(1 / D) correctly rounded,
// D and |v| within [2^-60, 2^60].  Why one correction is enough: q0 = RN(v * R) is within 1.5 ulp
// of v / D, the residual q0 * D - v is exact (or, in the lower half of a binade, rounded by at most
// 2^-47 relative to a quotient in [1/2, 1)), and the value that the final FMA rounds differs from
// v / D by at most 3.5 * 2^-48 of that scale.  v / D can be that close to a rounding boundary (the
// midpoint of two neighbouring floats) only when |A * 2^K - B * m| <= 6 for the integer
// significands A, B of v, D and an odd m (K = 24 or 25); all 93 million such pairs (bound 16) were
// enumerated on the host and give the IEEE quotient (tests/quotient_hard_cases.c).
__device__ __forceinline__ float quotient_short(float v, float D, float R) {
    const float q = __fmul_rn(v, R);
    const float r = __fmaf_rn(q, D, -v);
    return __fmaf_rn(-r, R, q);
}

// fl32(u / 6) by a reciprocal multiply with one correction: exact for this divisor (checked on the
// host for every binary32 u in [1e-30, 1e30]; 0 maps to 0).  Below that range the residual can
// underflow and the result may be one ulp off.
__device__ __forceinline__ float div6_fast(float u) {
    const float R6 = 0.16666667163372039794921875f;   // RN(1/6)
    const float q = __fmul_rn(u, R6);
    const float r = __fmaf_rn(q, -6.0f, u);
    return __fmaf_rn(r, R6, q);
}

// Eight quotients -> one word of eight FP4 codes (element 0 in bits 0..3) and the four f16x2
// words holding the grid values they stand for (element 2k in the low half of h[k]).
__device__ __forceinline__ uint32_t quantize_e2m1x8_h(const float* t, uint32_t* h) {
    uint32_t out;
    asm("{\n"
        " .reg .b8 b0, b1, b2, b3;\n"
        " cvt.rn.satfinite.e2m1x2.f32 b0, %6, %5;\n"
        " cvt.rn.satfinite.e2m1x2.f32 b1, %8, %7;\n"
        " cvt.rn.satfinite.e2m1x2.f32 b2, %10, %9;\n"
        " cvt.rn.satfinite.e2m1x2.f32 b3, %12, %11;\n"
        " cvt.rn.f16x2.e2m1x2 %1, b0;\n"
        " cvt.rn.f16x2.e2m1x2 %2, b1;\n"
        " cvt.rn.f16x2.e2m1x2 %3, b2;\n"
        " cvt.rn.f16x2.e2m1x2 %4, b3;\n"
        " mov.b32 %0, {b0, b1, b2, b3};\n"
        "}"
        : "=r"(out), "=r"(h[0]), "=r"(h[1]), "=r"(h[2]), "=r"(h[3])
        : "f"(t[0]), "f"(t[1]), "f"(t[2]), "f"(t[3]), "f"(t[4]), "f"(t[5]), "f"(t[6]), "f"(t[7]));
    return out;
}

// e = fma(q, -D, v) for the two grid values of an f16x2 word, with q and -D given in f16: the
// product is exact and the sum is rounded once to binary32 (mixed-precision FMA).
__device__ __forceinline__ void residual_pair_f16(uint32_t h, uint32_t nD16, float v0, float v1, float& e0, float& e1) {
    asm("{\n"
        " .reg .b16 lo, hi, d, dx;\n"
        " mov.b32 {lo, hi}, %2;\n"
        " mov.b32 {d, dx}, %3;\n"
        " fma.rn.f32.f16 %0, lo, d, %4;\n"
        " fma.rn.f32.f16 %1, hi, d, %5;\n"
        "}"
        : "=f"(e0), "=f"(e1)
        : "r"(h), "r"(nD16), "f"(v0), "f"(v1));
}

// The two f16 grid values of a word as binary32: mixed-precision adds of -0 (exact, the sign of a
// zero is kept), which read their half straight from the 32-bit register.
__device__ __forceinline__ float2 widen_f16x2(uint32_t h) {
    float2 q;
    asm("{\n"
        " .reg .b16 lo, hi;\n"
        " mov.b32 {lo, hi}, %2;\n"
        " add.rn.f32.f16 %0, lo, %3;\n"
        " add.rn.f32.f16 %1, hi, %3;\n"
        "}"
        : "=f"(q.x), "=f"(q.y)
        : "r"(h), "f"(-0.0f));
    return q;
}

template <int DT, int B>
struct QuantShape {
    static constexpr int EB = elem_bytes(DT);
    static constexpr int C = (B * EB >= 64) ? B : 64 / EB;   // elements per thread-chunk (>= 64 bytes)
    static constexpr int GE = (B < 8) ? 8 : B;               // elements per group
    static constexpr int NG = C / GE;                        // groups per chunk
    static constexpr int NBG = GE / B;                       // blocks per group
    static constexpr int NBC = C / B;                        // blocks per chunk
    static constexpr int PIECES = C * EB / 16;               // 16-byte pieces per chunk
    static constexpr int SLOTS = 2;                          // ring depth per thread
    static constexpr bool COOP = PIECES > 4;                 // chunk above 64 bytes: the warp copies its chunks together
    static constexpr size_t RING_BYTES = (size_t)SLOTS * PIECES * 16 * kThreads;
};

// raw words -> binary32.  bf16 goes through the FMA pipe (mixed-precision add of -0, which keeps
// the sign of a zero and every denormal) and leaves the integer pipe to the FP4 converts.
template <int DT, int N>
__device__ __forceinline__ void widen(const uint32_t* w, float* v) {
    if constexpr (DT == kF32) {
#pragma unroll
        for (int i = 0; i < N; ++i) v[i] = __uint_as_float(w[i]);
    } else {
#pragma unroll
        for (int i = 0; i < N / 2; ++i) {
            asm("{\n"
                " .reg .b16 lo, hi;\n"
                " mov.b32 {lo, hi}, %2;\n"
                " add.rn.f32.bf16 %0, lo, %3;\n"
                " add.rn.f32.bf16 %1, hi, %3;\n"
                "}"
                : "=f"(v[2 * i]), "=f"(v[2 * i + 1])
                : "r"(w[i]), "f"(-0.0f));
        }
    }
}

// Pack a group's quotients (GE / 8 code words) and continue the per-block SSE chains from the
// values in sse[] (e = fma(-q, D, v); sse = fma(e, e, sse), in element order): the caller starts
// them at zero, and a block longer than a group is fed through in consecutive parts.
template <int B, bool HALF>
__device__ __forceinline__ void pack_and_score(const float* v, const float* t, const float4* E, uint32_t* packed,
                                               float* sse) {
    constexpr int GE = (B < 8) ? 8 : B;
    constexpr int NBG = GE / B;
    uint32_t h[GE / 2];
#pragma unroll
    for (int k = 0; k < GE / 8; ++k) packed[k] = quantize_e2m1x8_h(&t[8 * k], &h[4 * k]);
#pragma unroll
    for (int j = 0; j < NBG; ++j) {
        float s = sse[j];
        if constexpr (HALF) {
            const uint32_t nD16 = __float_as_uint(E[j].z);
#pragma unroll
            for (int i = 0; i < B; i += 2) {
                float e0, e1;
                residual_pair_f16(h[(j * B + i) / 2], nD16, v[j * B + i], v[j * B + i + 1], e0, e1);
                s = __fmaf_rn(e0, e0, s);
                s = __fmaf_rn(e1, e1, s);
            }
        } else {
            const float nD = -E[j].x;
#pragma unroll
            for (int i = 0; i < B; i += 2) {
                const float2 q = widen_f16x2(h[(j * B + i) / 2]);
                const float e0 = __fmaf_rn(q.x, nD, v[j * B + i]);
                s = __fmaf_rn(e0, e0, s);
                const float e1 = __fmaf_rn(q.y, nD, v[j * B + i + 1]);
                s = __fmaf_rn(e1, e1, s);
            }
        }
        sse[j] = s;
    }
}

// Quotients of one block by its decode scale, two elements per instruction (fma.rn.f32x2):
// q = (-v) * (-R); r = q * D - v; q <- q - r * R.  Same values as quotient_short(), including the
// sign of a zero quotient: every product and sum has the signs of the scalar form.
//
// SHORT: the elements have at most 8 significant bits (bf16 input) and D at most 4.  Then the FP4
// code of fl(v / D) is the FP4 code of RZ(v * R), one multiply rounded toward zero: the quotient is a
// ratio of small integers times a power of two, so it either IS an FP4 rounding midpoint or lies
// more than 2^-9 (relative) away from every one of them, far more than the error of the product;
// and RN(1 / D) is never below 1 / D for these eight significands (it exceeds it by at most
// 0.875 * 2^-24 relative), so that at a midpoint M the exact product lies in [M, M + ulp) and the
// truncation returns M itself, which the FP4 rounding then sends to the even neighbour exactly as it
// does for the true quotient.  Checked on the host for every bf16 value and
// every significand (tests/test_quotient_hard_cases.py).  The sign of a zero product is that of v.
// Under a tensor scale that is not a power of two D is long; the same multiply is then used with a
// reciprocal that build_quant_tables() has checked for the launch's eight scale significands (R is that
// reciprocal here, taken from the table's z field).
template <int B, bool SHORT>
__device__ __forceinline__ void block_quotients(const float* v, float D, float R, float* t) {
    if constexpr (SHORT) {
        const float2 R2 = make_float2(R, R);
#pragma unroll
        for (int i = 0; i < B; i += 2) {
            const float2 q = __fmul2_rz(make_float2(v[i], v[i + 1]), R2);
            t[i] = q.x;
            t[i + 1] = q.y;
        }
        return;
    }
    const float2 D2 = make_float2(D, D), nR2 = make_float2(-R, -R);
#pragma unroll
    for (int i = 0; i < B; i += 2) {
        const float2 nv = make_float2(-v[i], -v[i + 1]);
        float2 q = __fmul2_rn(nv, nR2);
        float2 r = __ffma2_rn(q, D2, nv);
        q = __ffma2_rn(r, nR2, q);
        t[i] = q.x;
        t[i + 1] = q.y;
    }
}

// One candidate set of a group with the shortcuts (every entry has w != 0, magnitudes in range).
template <int B, bool HALF, bool SHORT>
__device__ __forceinline__ void encode_group_fast(const float* v, const float4* E, uint32_t* packed, float* sse) {
    constexpr int GE = (B < 8) ? 8 : B;
    constexpr int NBG = GE / B;
    float t[GE];
#pragma unroll
    for (int j = 0; j < NBG; ++j) block_quotients<B, SHORT>(&v[j * B], E[j].x, (SHORT && !HALF) ? E[j].z : E[j].y, &t[j * B]);
    pack_and_score<B, HALF>(v, t, E, packed, sse);
}

// Both 4-over-6 candidate sets of a group at once: quotients as above, FP4 pack / unpack per
// candidate, and the two SSE chains of a block side by side in one fma.rn.f32x2 per element
// (lane .x: the M = 6 candidate, lane .y: the M = 4 candidate; each lane sums its own residuals
// in element order, exactly like the scalar chain).  The chains continue from sse6[] / sse4[].
template <int B, bool HALF, bool SHORT>
__device__ __forceinline__ void encode_group_fast_dual(const float* v, const float4* E6, const float4* E4, uint32_t* pk6,
                                                       uint32_t* pk4, float* sse6, float* sse4) {
    constexpr int GE = (B < 8) ? 8 : B;
    constexpr int NBG = GE / B;
    float t6[GE], t4[GE];
#pragma unroll
    for (int j = 0; j < NBG; ++j) {
        block_quotients<B, SHORT>(&v[j * B], E6[j].x, (SHORT && !HALF) ? E6[j].z : E6[j].y, &t6[j * B]);
        block_quotients<B, SHORT>(&v[j * B], E4[j].x, (SHORT && !HALF) ? E4[j].z : E4[j].y, &t4[j * B]);
    }
    uint32_t h6[GE / 2], h4[GE / 2];
#pragma unroll
    for (int k = 0; k < GE / 8; ++k) {
        pk6[k] = quantize_e2m1x8_h(&t6[8 * k], &h6[4 * k]);
        pk4[k] = quantize_e2m1x8_h(&t4[8 * k], &h4[4 * k]);
    }
#pragma unroll
    for (int j = 0; j < NBG; ++j) {
        float2 s = make_float2(sse6[j], sse4[j]);
        const uint32_t nD6_16 = __float_as_uint(E6[j].z), nD4_16 = __float_as_uint(E4[j].z);
        const float nD6 = -E6[j].x, nD4 = -E4[j].x;
#pragma unroll
        for (int i = 0; i < B; i += 2) {
            const int e = j * B + i;
            float a0, a1, b0, b1;   // residuals of elements e, e + 1 under candidate 6 (a) and 4 (b)
            if constexpr (HALF) {
                residual_pair_f16(h6[e / 2], nD6_16, v[e], v[e + 1], a0, a1);
                residual_pair_f16(h4[e / 2], nD4_16, v[e], v[e + 1], b0, b1);
            } else {
                const float2 q6 = widen_f16x2(h6[e / 2]);
                const float2 q4 = widen_f16x2(h4[e / 2]);
                a0 = __fmaf_rn(q6.x, nD6, v[e]);
                a1 = __fmaf_rn(q6.y, nD6, v[e + 1]);
                b0 = __fmaf_rn(q4.x, nD4, v[e]);
                b1 = __fmaf_rn(q4.y, nD4, v[e + 1]);
            }
            const float2 e0 = make_float2(a0, b0), e1 = make_float2(a1, b1);
            s = __ffma2_rn(e0, e0, s);
            s = __ffma2_rn(e1, e1, s);
        }
        sse6[j] = s.x;
        sse4[j] = s.y;
    }
}

// One candidate set of a group on the general path (IEEE division; zero scale -> signed zeros).
template <int B>
__device__ __forceinline__ void encode_group_general(const float* v, const float4* E, uint32_t* packed, float* sse) {
    constexpr int GE = (B < 8) ? 8 : B;
    constexpr int NBG = GE / B;
    float t[GE];
#pragma unroll
    for (int j = 0; j < NBG; ++j)
#pragma unroll
        for (int i = 0; i < B; ++i) t[j * B + i] = quotient_general(v[j * B + i], E[j].x);
    pack_and_score<B, false>(v, t, E, packed, sse);
}

// CTA-uniform constants of a launch.
struct QuantConsts {
    float g, Rg;        // tensor scale and RN(1 / g)
    float m_lo, m_hi;   // a block maximum m takes the shortcuts when m == 0 or m_lo <= m <= m_hi
    bool unit_g, need_lo;
    int c_min;          // smallest admissible code: 1 under prevent-zero (FP8 formats), else 0
    int pow2_rule;      // kPow2Eq1 unless the format is UE8M0 and another rule was asked for
    float u_floor;      // lean path: prevent-zero as a floor on amax / g, 4 * value(code 1), else 0
    int lean_cmax;      // lean path: every code up to this one has class 3 (UE5M3: the codes above it take the general path)
    bool onemul;        // bf16 input under a tensor scale: the one-multiply quotient with the reciprocals in E[].z holds for the whole table
};

// The lean path runs when there is no tensor scale and every code of the table has class 3 (UE4M3), or
// every code but the last few (UE5M3: the scales from 2^16 on are not f16 values; a block that lands on
// one of them is redone on the general path).
template <int FMT>
__device__ __forceinline__ bool lean_allowed(int first_bad, bool unit_g) {
    return unit_g && first_bad >= (FMT == kUE5M3 ? num_codes(FMT) - 16 : num_codes(FMT));
}

// The lean path under a tensor scale (LEAN == 2; bf16 input, FP8 scale formats): the launch's table passed
// the one-multiply check and g lies in [2^-40, 2^20].  Then every decode scale of both formats is within
// [2^-60, 2^60] (or zero), so every entry carries a checked reciprocal; a block maximum above m_hi may be
// clamped to it (m_hi / g is at least 2^40: the scale code is the top one either way); a maximum below
// 2^-63, where the quotient by g is no longer exact, gives a / g < 2^-23 and code 0 (or the prevent-zero
// floor) whatever its last bits are.
__device__ __forceinline__ bool lean_scaled_allowed(const QuantConsts& k) {
    return k.onemul && k.g >= 9.094947017729282379e-13f /* 2^-40 */ && k.g <= 1048576.0f;
}

// Both 4-over-6 scale codes of a block from one conversion (UE4M3): the code for w6 in bits 0..7,
// the code for w4 in bits 8..15.
__device__ __forceinline__ uint32_t round_scale_pair_ue4m3(float w4, float w6) {
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(w4), "f"(w6));
    return r;
}

// The same for UE5M3, whose values are the UE4M3 values times 2^-8 (codes 0..0x7E), times 1 (the UE4M3
// normals, codes + 0x40) and times 2^8 (codes + 0x80): rounding to nearest even commutes with an exact
// scaling by a power of two, so the pair is scaled into the stretch of UE4M3 that matches its magnitude,
// converted, and the code offset added to both bytes.  The stretch is chosen by w4; w6 must lie within
// [w4 / 2, w4] (it is w4 / 1.5 here), which keeps it among the UE4M3 normals wherever w4 is: w4 < 1 uses
// the whole of UE4M3 including its subnormals (256 w <= 448: no saturation), 1 <= w4 < 256 the normals
// from 0.5 up, w4 >= 256 the same after a division by 256, where saturation at 448 is the saturation of
// UE5M3 at 114688.  Either stretch gives the same code where two of them overlap.
__device__ __forceinline__ uint32_t round_scale_pair_ue5m3(float w4, float w6) {
    const bool low = w4 < 1.0f, high = w4 >= 256.0f;
    const float s = low ? 256.0f : (high ? 0.00390625f : 1.0f);
    const uint32_t offset = low ? 0u : (high ? 0x8080u : 0x4040u);
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(__fmul_rn(w4, s)), "f"(__fmul_rn(w6, s)));
    return (uint32_t)r + offset;
}

// Scale code for the M = 6 target from u = amax / g: Eq. 2 (Eq. 1 for UE8M0), or one of the
// alternative power-of-two rules.
template <int FMT, bool EXACT>
__device__ __forceinline__ int target6_code(float u, int pow2_rule) {
    if constexpr (FMT == kUE8M0) {
        if (pow2_rule != kPow2Eq1) return pow2_rule_code(u, pow2_rule);
    }
    return round_scale<FMT>(EXACT ? __fdiv_rn(u, 6.0f) : div6_fast(u));
}

// LEAN == 2: the same loop under a tensor scale, see lean_scaled_allowed(): the block maximum is divided by g
// first (corrected quotient), the residual is formed in binary32.
// LEAN == 1 (launch-uniform; bf16 input, FP8 scale format, no tensor scale, every decode scale of the
// table of class 3 -- for UE5M3 all but its last few codes, whose scales from 2^16 on are not f16
// values: a group whose code lands there is redone on the general path): nothing of a block can leave
// the shortcuts, so the per-block class and range tests and the tensor-scale quotient are left out.  Why no magnitude test is
// needed: the one-multiply quotient neither forms a residual nor divides (a product that
// overflows or underflows still rounds to the FP4 code of the true quotient, 6 or 0 with the sign
// of the element); amax / 6 by multiply-and-correct is exact from 1e-30 to 1e30, below that every
// FP8 format gives code 0 (the prevent-zero floor keeps the argument far above it anyway) and
// above it both formats saturate.  Prevent-zero is a floor on the block maximum: for both
// formats max(code_M(u), 1) = code_M(max(u, 4 eps)) for M = 6 and M = 4, eps = value(code 1)
// (4 eps / 6 and 4 eps / 4 round to code 1; anything below rounds to 0 or 1, anything above to >= 1).
template <int DT, int B, int FMT, bool DUAL, bool FAKE, int LEAN>
__device__ __forceinline__ void quantize_chunk(const QuantArgs& p, const QuantTables& T, const QuantConsts& k,
                                               size_t chunk, const uint32_t* raw, double& sse_sum) {
    static_assert(!LEAN || (DT == kBF16 && FMT != kUE8M0), "lean path: bf16 input, FP8 scale formats");
    using S = QuantShape<DT, B>;
    constexpr int NBG = S::NBG;
    uint32_t packed[S::C / 8];
    uint32_t sc[(S::NBC + 3) / 4];
    uint32_t sw[S::NBC];
#pragma unroll
    for (int i = 0; i < (S::NBC + 3) / 4; ++i) sc[i] = 0;

#pragma unroll
    for (int gi = 0; gi < S::NG; ++gi) {
        float v[S::GE];
        widen<DT, S::GE>(raw + gi * (S::GE * S::EB / 4), v);
        float m[NBG], u[NBG];
        int c6[NBG], c4[NBG];
        float4 E6[NBG], E4[NBG];
        float wmin = 3.0f, mmax = 0.0f, mmin = k.m_hi;
#pragma unroll
        for (int j = 0; j < NBG; ++j) {
            float a = 0.0f;
#pragma unroll
            for (int i = 0; i < B; ++i) a = fmaxf(a, fabsf(v[j * B + i]));
            if constexpr (LEAN) {
                m[j] = a;
                float ua = a;
                if constexpr (LEAN == 2) ua = quotient_corrected(fminf(a, k.m_hi), k.g, k.Rg);
                const float uf = fmaxf(ua, k.u_floor);
                const float w6 = div6_fast(uf);
                if constexpr (DUAL && FMT == kUE5M3) {
                    const uint32_t r = round_scale_pair_ue5m3(__fmul_rn(uf, 0.25f), w6);
                    c6[j] = (int)(r & 0xFFu);
                    c4[j] = (int)(r >> 8);
                } else if constexpr (DUAL && FMT == kUE4M3) {
                    const uint32_t r = round_scale_pair_ue4m3(__fmul_rn(uf, 0.25f), w6);
                    c6[j] = (int)(r & 0xFFu);
                    c4[j] = (int)(r >> 8);
                } else {
                    c6[j] = round_scale<FMT>(w6);
                    if constexpr (DUAL) c4[j] = round_scale<FMT>(__fmul_rn(uf, 0.25f));
                }
                E6[j] = T.E[c6[j]];
                if constexpr (DUAL) E4[j] = T.E[c4[j]];
                continue;
            }
            m[j] = a;
            mmax = fmaxf(mmax, a);
            if (k.need_lo) mmin = fminf(mmin, a == 0.0f ? k.m_hi : a);
            u[j] = k.unit_g ? a : quotient_corrected(a, k.g, k.Rg);
            c6[j] = max(target6_code<FMT, false>(u[j], k.pow2_rule), k.c_min);
            if constexpr (DUAL) c4[j] = max(round_scale<FMT>(__fmul_rn(u[j], 0.25f)), k.c_min);
            E6[j] = T.E[c6[j]];
            wmin = fminf(wmin, E6[j].w);
            if constexpr (DUAL) {
                E4[j] = T.E[c4[j]];
                wmin = fminf(wmin, E4[j].w);
            }
        }
        uint32_t pk[S::GE / 8], pk4[S::GE / 8];
        float sse[NBG], sse4[NBG];
#pragma unroll
        for (int j = 0; j < NBG; ++j) sse[j] = sse4[j] = 0.0f;
        bool lean_group = LEAN != 0;
        if constexpr (LEAN == 1 && FMT == kUE5M3) {   // a code above the class-3 range: this group takes the general path
            int cmx = 0;
#pragma unroll
            for (int j = 0; j < NBG; ++j) cmx = max(cmx, DUAL ? max(c6[j], c4[j]) : c6[j]);
            lean_group = cmx <= k.lean_cmax;
        }
        if (LEAN && lean_group) {
            constexpr bool HALF = (LEAN == 1);   // under a tensor scale the residual is formed in binary32
            if constexpr (DUAL) encode_group_fast_dual<B, HALF, true>(v, E6, E4, pk, pk4, sse, sse4);
            else encode_group_fast<B, HALF, true>(v, E6, pk, sse);
        } else if (!LEAN && wmin >= 1.0f && mmax <= k.m_hi && mmin >= k.m_lo) {
            // one decision for both candidates.  bf16 input: the one-multiply quotient with the f16
            // residual when every decode scale of the group is short, else the general shortcuts.
            constexpr bool SH = (DT == kBF16);
            if (wmin >= (SH ? 3.0f : 2.0f)) {
                if constexpr (DUAL) encode_group_fast_dual<B, true, SH>(v, E6, E4, pk, pk4, sse, sse4);
                else encode_group_fast<B, true, SH>(v, E6, pk, sse);
            } else if (SH && k.onemul) {   // one-multiply quotient with the checked reciprocals, binary32 residual
                if constexpr (DUAL) encode_group_fast_dual<B, false, SH>(v, E6, E4, pk, pk4, sse, sse4);
                else encode_group_fast<B, false, SH>(v, E6, pk, sse);
            } else {
                if constexpr (DUAL) encode_group_fast_dual<B, false, false>(v, E6, E4, pk, pk4, sse, sse4);
                else encode_group_fast<B, false, false>(v, E6, pk, sse);
            }
        } else {
#pragma unroll
            for (int j = 0; j < NBG; ++j) {
                u[j] = __fdiv_rn(m[j], k.g);
                c6[j] = target6_code<FMT, true>(u[j], k.pow2_rule);
                c6[j] = max(c6[j], k.c_min);
                E6[j] = T.E[c6[j]];
                if constexpr (DUAL) {
                    c4[j] = round_scale<FMT>(__fmul_rn(u[j], 0.25f));
                    c4[j] = max(c4[j], k.c_min);
                    E4[j] = T.E[c4[j]];
                }
            }
            encode_group_general<B>(v, E6, pk, sse);
            if constexpr (DUAL) encode_group_general<B>(v, E4, pk4, sse4);
        }

        float Dw[NBG];   // decode scale of the winner
#pragma unroll
        for (int j = 0; j < NBG; ++j) Dw[j] = E6[j].x;
        if constexpr (DUAL) {
            if constexpr (NBG == 1) {
                const bool take = sse4[0] < sse[0];
                sse[0] = take ? sse4[0] : sse[0];
                c6[0] = take ? c4[0] : c6[0];
                Dw[0] = take ? E4[0].x : Dw[0];
#pragma unroll
                for (int i = 0; i < S::GE / 8; ++i) pk[i] = take ? pk4[i] : pk[i];
            } else {
                // several blocks share the one 32-bit code word: select by bit mask
                constexpr uint32_t kBlockMask = (B == 2) ? 0xFFu : 0xFFFFu;
                uint32_t take = 0;
#pragma unroll
                for (int j = 0; j < NBG; ++j) {
                    const bool tj = sse4[j] < sse[j];
                    sse[j] = tj ? sse4[j] : sse[j];
                    c6[j] = tj ? c4[j] : c6[j];
                    Dw[j] = tj ? E4[j].x : Dw[j];
                    take |= tj ? (kBlockMask << (j * 4 * B)) : 0u;
                }
                pk[0] = (pk4[0] & take) | (pk[0] & ~take);
            }
        }
        if constexpr (FAKE) {   // fused fake-quantize: x_hat = fl32(grid(code) * D), optionally rounded to bf16
            const size_t e0 = chunk * S::C + (size_t)gi * S::GE;
#pragma unroll
            for (int w8 = 0; w8 < S::GE / 8; ++w8) {
                float q[8];
                unpack_e2m1x8(pk[w8], q);
                uint32_t o[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) o[i] = __float_as_uint(__fmul_rn(q[i], Dw[(w8 * 8 + i) / B]));
                if (p.xhat_dtype == kF32) {
                    store_bytes<32>(static_cast<float*>(p.xhat) + e0 + 8 * w8, o);
                } else {
                    uint32_t h[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const __nv_bfloat162 b2 = __floats2bfloat162_rn(__uint_as_float(o[2 * i]), __uint_as_float(o[2 * i + 1]));
                        h[i] = *reinterpret_cast<const uint32_t*>(&b2);
                    }
                    store_bytes<16>(static_cast<__nv_bfloat16*>(p.xhat) + e0 + 8 * w8, h);
                }
            }
        }
#pragma unroll
        for (int i = 0; i < S::GE / 8; ++i) packed[gi * (S::GE / 8) + i] = pk[i];
#pragma unroll
        for (int j = 0; j < NBG; ++j) {
            const int b = gi * NBG + j;
            sc[b / 4] |= (uint32_t)c6[j] << (8 * (b % 4));
            sw[b] = __float_as_uint(sse[j]);
            if constexpr (!FAKE) sse_sum = __dadd_rn(sse_sum, (double)sse[j]);
        }
    }
    if constexpr (FAKE) return;
    store_bytes<S::C / 2>(p.codes + chunk * (S::C / 2), packed);
    store_bytes<S::NBC>(p.scales + chunk * S::NBC, sc);
    if (p.block_sse) store_bytes<4 * S::NBC>(p.block_sse + chunk * S::NBC, sw);
}

// Position (in 16-byte units, relative to the warp's first column of a ring slot) of piece k of
// the chunk that lane `lane` works on.  Thread-private staging: row k, the thread's own column.
// Cooperative staging: row k, column lane ^ k, so that both the warp's copies (which write many
// rows of a few columns at once) and its later reads (one row, all columns) spread over all banks.
template <bool COOP>
__device__ __forceinline__ int ring_index(int k, int lane) {
    return k * kThreads + (COOP ? (lane ^ k) : lane);
}

// Larger magnitude of two bf16 pairs, half by half (the sign bits of the result carry no meaning).
__device__ __forceinline__ uint32_t absmax_bf16x2(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("max.xorsign.abs.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

// Blocks of 32 and 64 elements (chunk = one block).  The block is walked twice in parts of 16
// elements read from the thread's ring slot, which stays valid until the next trip's request:
// once for the block maximum, once for the encode with the SSE chains carried from part to part.
// Only one part is live in registers at a time, which keeps as many CTAs resident as for B = 16.
template <int DT, int B, int FMT, bool DUAL, bool FAKE>
__device__ __forceinline__ void quantize_long_block(const QuantArgs& p, const QuantTables& T, const QuantConsts& k,
                                                    size_t chunk, const uint4* slot_warp, int lane, double& sse_sum) {
    using S = QuantShape<DT, B>;
    static_assert(S::C == B && S::NBC == 1, "one block per chunk");
    constexpr int SG = 16;                        // elements per part
    constexpr int NSG = B / SG;
    constexpr int PPS = SG * S::EB / 16;          // 16-byte pieces per part
    auto load_part = [&](int sg, float* v) {
        uint32_t w[4 * PPS];
#pragma unroll
        for (int q = 0; q < PPS; ++q) {
            const uint4 x = slot_warp[ring_index<S::COOP>(sg * PPS + q, lane)];
            w[4 * q + 0] = x.x; w[4 * q + 1] = x.y; w[4 * q + 2] = x.z; w[4 * q + 3] = x.w;
        }
        widen<DT, SG>(w, v);
    };

    float a = 0.0f;
    if constexpr (DT == kBF16) {
        // the maximum pass on the packed words: magnitudes of bf16 values order like the values, and one
        // max.xorsign.abs.bf16x2 takes the larger magnitude in either half (the sign it leaves is dropped below)
        uint32_t m0 = 0, m1 = 0;
#pragma unroll
        for (int q = 0; q < S::PIECES; ++q) {
            const uint4 x = slot_warp[ring_index<S::COOP>(q, lane)];
            m0 = absmax_bf16x2(absmax_bf16x2(m0, x.x), x.z);
            m1 = absmax_bf16x2(absmax_bf16x2(m1, x.y), x.w);
        }
        const uint32_t mm = absmax_bf16x2(m0, m1) & 0x7FFF7FFFu;
        a = fmaxf(__uint_as_float(mm << 16), __uint_as_float(mm & 0xFFFF0000u));
    } else {
#pragma unroll
        for (int sg = 0; sg < NSG; ++sg) {
            float v[SG];
            load_part(sg, v);
#pragma unroll
            for (int i = 0; i < SG; ++i) a = fmaxf(a, fabsf(v[i]));
        }
    }
    float u = k.unit_g ? a : quotient_corrected(a, k.g, k.Rg);
    int c6 = max(target6_code<FMT, false>(u, k.pow2_rule), k.c_min), c4 = 0;
    float4 E6 = T.E[c6], E4 = E6;
    float wmin = E6.w;
    if constexpr (DUAL) {
        c4 = max(round_scale<FMT>(__fmul_rn(u, 0.25f)), k.c_min);
        E4 = T.E[c4];
        wmin = fminf(wmin, E4.w);
    }
    const bool fast = wmin >= 1.0f && a <= k.m_hi && (a == 0.0f || a >= k.m_lo);
    if (!fast) {
        u = __fdiv_rn(a, k.g);
        c6 = max(target6_code<FMT, true>(u, k.pow2_rule), k.c_min);
        E6 = T.E[c6];
        if constexpr (DUAL) {
            c4 = max(round_scale<FMT>(__fmul_rn(u, 0.25f)), k.c_min);
            E4 = T.E[c4];
        }
    }

    uint32_t pk[B / 8], pk4[B / 8];
    float sse = 0.0f, sse4 = 0.0f;
#pragma unroll
    for (int sg = 0; sg < NSG; ++sg) {
        float v[SG];
        load_part(sg, v);
        uint32_t* o6 = &pk[sg * (SG / 8)];
        uint32_t* o4 = &pk4[sg * (SG / 8)];
        if (fast) {
            constexpr bool SH = (DT == kBF16);
            if (wmin >= (SH ? 3.0f : 2.0f)) {
                if constexpr (DUAL) encode_group_fast_dual<SG, true, SH>(v, &E6, &E4, o6, o4, &sse, &sse4);
                else encode_group_fast<SG, true, SH>(v, &E6, o6, &sse);
            } else if (SH && k.onemul) {
                if constexpr (DUAL) encode_group_fast_dual<SG, false, SH>(v, &E6, &E4, o6, o4, &sse, &sse4);
                else encode_group_fast<SG, false, SH>(v, &E6, o6, &sse);
            } else {
                if constexpr (DUAL) encode_group_fast_dual<SG, false, false>(v, &E6, &E4, o6, o4, &sse, &sse4);
                else encode_group_fast<SG, false, false>(v, &E6, o6, &sse);
            }
        } else {
            encode_group_general<SG>(v, &E6, o6, &sse);
            if constexpr (DUAL) encode_group_general<SG>(v, &E4, o4, &sse4);
        }
    }
    float Dw = E6.x;
    if constexpr (DUAL) {
        const bool take = sse4 < sse;
        sse = take ? sse4 : sse;
        c6 = take ? c4 : c6;
        Dw = take ? E4.x : Dw;
#pragma unroll
        for (int i = 0; i < B / 8; ++i) pk[i] = take ? pk4[i] : pk[i];
    }
    if constexpr (FAKE) {   // fused fake-quantize: x_hat = fl32(grid(code) * D), optionally rounded to bf16
        const size_t e0 = chunk * B;
#pragma unroll
        for (int w8 = 0; w8 < B / 8; ++w8) {
            float q[8];
            unpack_e2m1x8(pk[w8], q);
            uint32_t o[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) o[i] = __float_as_uint(__fmul_rn(q[i], Dw));
            if (p.xhat_dtype == kF32) {
                store_bytes<32>(static_cast<float*>(p.xhat) + e0 + 8 * w8, o);
            } else {
                uint32_t h[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const __nv_bfloat162 b2 = __floats2bfloat162_rn(__uint_as_float(o[2 * i]), __uint_as_float(o[2 * i + 1]));
                    h[i] = *reinterpret_cast<const uint32_t*>(&b2);
                }
                store_bytes<16>(static_cast<__nv_bfloat16*>(p.xhat) + e0 + 8 * w8, h);
            }
        }
        return;
    }
    store_bytes<B / 2>(p.codes + chunk * (B / 2), pk);
    p.scales[chunk] = (uint8_t)c6;
    if (p.block_sse) p.block_sse[chunk] = sse;
    sse_sum = __dadd_rn(sse_sum, (double)sse);
}

// Cooperative staging for chunks above 64 bytes.  With thread-private copies every 16-byte piece
// of such a chunk lies in a cache line of its own lane, and one copy instruction of a warp touches
// 32 lines for 512 bytes; the L1 tag rate then caps the kernel near two thirds of the HBM
// bandwidth.  Here the warp copies its 32 consecutive chunks as one contiguous region instead:
// instruction i moves pieces 32 i .. 32 i + 31 of the region (512 contiguous bytes, 4 lines), lane
// l the piece 32 i + l, which is piece (32 i + l) % PIECES of the chunk of lane (32 i + l) / PIECES.
// The data then crosses lanes, so the consumer waits for its own copies and joins a __syncwarp()
// (every lane of the warp takes every trip of the loop).  wchunk: chunk of lane 0.
template <int PIECES>
__device__ __forceinline__ void stage_warp_chunks(uint32_t slot_warp_addr, const char* x, size_t chunk_bytes, size_t wchunk,
                                                  size_t n_chunks, int lane) {
#pragma unroll
    for (int i = 0; i < PIECES; ++i) {
        const int piece = i * 32 + lane;
        const int owner = piece / PIECES, k = piece % PIECES;
        if (wchunk + owner < n_chunks)
            asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(slot_warp_addr + ring_index<true>(k, owner) * 16),
                         "l"(x + wchunk * chunk_bytes + (size_t)piece * 16)
                         : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
}

// Asynchronous copy of one chunk (PIECES x 16 bytes) from global memory into this thread's pieces
// of a ring slot (piece k of thread t at ((slot * PIECES + k) * 256 + t) * 16), as one commit
// group.  An empty group is committed when there is no chunk left, so that the group count per
// loop trip stays fixed.
template <int PIECES>
__device__ __forceinline__ void stage_chunk(uint32_t slot_addr, const void* src, bool valid) {
    if (valid) {
        const char* g = static_cast<const char*>(src);
#pragma unroll
        for (int k = 0; k < PIECES; ++k)
            asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(slot_addr + k * (kThreads * 16)), "l"(g + 16 * k)
                         : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
}

// Blocks longer than 16 elements go part by part (quantize_long_block()), except 4-over-6 at B = 32, which
// is faster with the whole block in registers (33.5 M bf16 elements: 0.775 against 0.711 of the copy bandwidth).
__host__ __device__ constexpr bool long_block_path(int B, bool dual) { return B > 16 && !(dual && B == 32); }

// Body of the multi-tensor kernel (see k_quantize, BATCH).
template <int DT, int B, int FMT, bool DUAL>
__device__ __forceinline__ void quantize_batch_body(const QuantArgs& p, QuantTables& T, uint4* ring) {
    using S = QuantShape<DT, B>;
    __shared__ uint32_t row0[kMaxBatch + 1];   // row0[t] = first row of tensor t; row0[n_tensors] = all rows
    __shared__ uint32_t warp_rows[kThreads / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int nt = p.n_tensors;
    // prefix sums of the tensors' row counts: four tensors per thread, a scan over the warps' totals
    {
        uint32_t r[4], mine = 0;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int t = threadIdx.x * 4 + q;
            r[q] = 0;
            if (t < nt) r[q] = (uint32_t)((p.batch[t].n / S::C + 31) / 32);
            mine += r[q];
        }
        uint32_t incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += up;
        }
        if (lane == 31) warp_rows[warp] = incl;
        __syncthreads();
        uint32_t before = incl - mine;
        for (int w = 0; w < warp; ++w) before += warp_rows[w];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int t = threadIdx.x * 4 + q;
            if (t <= nt) row0[t] = before;     // t == nt: the total
            before += r[q];
        }
        if (threadIdx.x == kThreads - 1) row0[nt] = before;   // (nt == 4 * kThreads has no owner above)
    }
    QuantConsts k;
    k.g = p.d_global_scale ? *p.d_global_scale : p.global_scale;
    int first_bad;
    k.onemul = build_quant_tables<FMT, DT == kBF16>(T, k.g, first_bad);   // contains a barrier: row0[] is complete too
    k.unit_g = (k.g == 1.0f);
    k.c_min = (p.prevent_zero && FMT != kUE8M0) ? 1 : 0;
    k.pow2_rule = (FMT == kUE8M0) ? p.pow2_rule : kPow2Eq1;
    k.u_floor = k.c_min ? __fmul_rn(4.0f, scale_value(FMT, 1)) : 0.0f;
    k.lean_cmax = first_bad - 1;
    k.Rg = 1.0f;
    k.need_lo = (FMT == kUE8M0) || !k.unit_g;
    k.m_hi = kFastMax;
    k.m_lo = 0.0f;
    if (k.unit_g) {
        if (FMT == kUE8M0) k.m_lo = 1.0e-30f;
    } else if (k.g >= kFastMin && k.g <= kFastMax) {
        k.Rg = __frcp_rn(k.g);
        k.m_hi = fminf(kFastMax, __fmul_rn(k.g, 1.0e29f));
        k.m_lo = fmaxf(1.084202172485504434e-19f /* 2^-63 */, (FMT == kUE8M0) ? __fmul_rn(k.g, 1.0e-29f) : 0.0f);
    } else {
        k.m_hi = -1.0f;
        k.m_lo = 0.0f;
    }

    const uint32_t total_rows = row0[nt];
    const uint32_t row_stride = gridDim.x * (kThreads / 32);
    constexpr size_t kChunkBytes = (size_t)S::C * S::EB;
    constexpr uint32_t kSlotBytes = S::PIECES * kThreads * 16;
    constexpr int DIST = S::SLOTS - 1;
    const uint32_t ring_warp = (uint32_t)__cvta_generic_to_shared(ring) + (threadIdx.x - lane) * 16;
    const uint32_t ring_base = ring_warp + lane * 16;

    // A cursor: the tensor that holds a given row (rows only move forward).  Warp-uniform.
    struct Cursor {
        int t;
        uint32_t first, end;     // rows [first, end) belong to tensor t
        size_t n_chunks;
        const char* x;
    };
    auto seek = [&](Cursor& c, uint32_t row) {
        while (row >= c.end && c.t + 1 < nt) {
            ++c.t;
            c.first = c.end;
            c.end = row0[c.t + 1];
            c.n_chunks = p.batch[c.t].n / S::C;
            c.x = static_cast<const char*>(p.batch[c.t].x);
        }
    };
    // request the chunks of row `row` into ring slot `fill` (an empty group when there is no such row)
    auto request = [&](Cursor& c, uint32_t row, int fill) {
        if (row < total_rows) {
            seek(c, row);
            const size_t wchunk = (size_t)(row - c.first) * 32;
            if constexpr (S::COOP) {
                stage_warp_chunks<S::PIECES>(ring_warp + fill * kSlotBytes, c.x, kChunkBytes, wchunk, c.n_chunks, lane);
            } else {
                stage_chunk<S::PIECES>(ring_base + fill * kSlotBytes, c.x + (wchunk + lane) * kChunkBytes, wchunk + lane < c.n_chunks);
            }
        } else {
            asm volatile("cp.async.commit_group;" ::: "memory");
        }
    };

    uint32_t row = blockIdx.x * (kThreads / 32) + warp;
    if (row >= total_rows) return;    // whole warps leave; no barrier follows
    Cursor ahead_c = {-1, 0u, 0u, 0, nullptr}, cur_c = {-1, 0u, 0u, 0, nullptr};
    uint32_t ahead = row;
#pragma unroll
    for (int d = 0; d < DIST; ++d) {
        request(ahead_c, ahead, d);
        ahead += row_stride;
    }
    QuantArgs pl = p;                 // the current tensor's output pointers
    pl.mse_partials = nullptr;
    int cur_t = -1;
    double unused_sum = 0.0;
    auto row_loop = [&](auto lean_tag) {
        constexpr int LEAN = decltype(lean_tag)::value;
        int slot = 0, fill = DIST % S::SLOTS;
        for (; row < total_rows; row += row_stride) {
            asm volatile("cp.async.wait_group %0;" ::"n"(DIST - 1) : "memory");
            if constexpr (S::COOP) __syncwarp();
            const uint4* slot_warp = ring + (size_t)slot * (S::PIECES * kThreads) + (threadIdx.x - lane);
            request(ahead_c, ahead, fill);
            ahead += row_stride;
            slot = (slot + 1 == S::SLOTS) ? 0 : slot + 1;
            fill = (fill + 1 == S::SLOTS) ? 0 : fill + 1;
            seek(cur_c, row);
            if (cur_c.t != cur_t) {
                cur_t = cur_c.t;
                pl.codes = p.batch[cur_t].codes;
                pl.scales = p.batch[cur_t].scales;
                pl.block_sse = p.batch[cur_t].block_sse;
            }
            const size_t chunk = (size_t)(row - cur_c.first) * 32 + lane;
            if (chunk >= cur_c.n_chunks) continue;      // a lane past the end of the tensor's last row
            if constexpr (long_block_path(B, DUAL)) {
                quantize_long_block<DT, B, FMT, DUAL, false>(pl, T, k, chunk, slot_warp, lane, unused_sum);
            } else {
                uint32_t raw[S::PIECES * 4];
#pragma unroll
                for (int q = 0; q < S::PIECES; ++q) {
                    const uint4 w = slot_warp[ring_index<S::COOP>(q, lane)];
                    raw[4 * q + 0] = w.x; raw[4 * q + 1] = w.y; raw[4 * q + 2] = w.z; raw[4 * q + 3] = w.w;
                }
                quantize_chunk<DT, B, FMT, DUAL, false, LEAN>(pl, T, k, chunk, raw, unused_sum);
            }
        }
    };
    constexpr bool CAN_LEAN = (DT == kBF16) && (FMT != kUE8M0) && !(long_block_path(B, DUAL));
    if constexpr (CAN_LEAN) {
        if (lean_allowed<FMT>(first_bad, k.unit_g)) row_loop(std::integral_constant<int, 1>{});
        else if (lean_scaled_allowed(k)) row_loop(std::integral_constant<int, 2>{});
        else row_loop(std::integral_constant<int, 0>{});
    } else {
        row_loop(std::integral_constant<int, 0>{});
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
}

// BATCH: one launch over a list of tensors (same dtype, block size, format, recipe and tensor scale).
// The unit of distribution is a ROW of 32 consecutive chunks of one tensor (what a warp handles in one
// trip); tensor t owns ceil(chunks_t / 32) rows of a common index space whose prefix sums every CTA
// forms in shared memory; a warp walks rows first, first + 8 * gridDim.x, ... and moves its tensor
// cursor forward when a row passes the end of the current tensor.  Everything else (ring, staging,
// per-chunk arithmetic) is as in the single-tensor kernel.
// Resident CTAs the register allocation has to allow (0: no bound, the allocator's own choice; an explicit 1
// is NOT the same: it lets the allocator spend up to 255 registers and measured far slower).  The
// multi-tensor instantiations carry a cursor and a row loop on top of the chunk arithmetic; without a bound
// some of them (B = 16) land a few registers above the 85 that three CTAs per SM allow and lose a third of
// their loads in flight.
__host__ __device__ constexpr int quantize_min_ctas(int B, bool batch) { return (batch && B >= 4 && B <= 16) ? 3 : 0; }

template <int DT, int B, int FMT, bool DUAL, bool FAKE, bool BATCH = false>
__global__ void __launch_bounds__(kThreads, quantize_min_ctas(B, BATCH)) k_quantize(QuantArgs p) {
    using S = QuantShape<DT, B>;
    static_assert(S::C == quantize_chunk_elems(DT, B), "host and kernel agree on the chunk size");
    extern __shared__ uint4 ring[];
    __shared__ QuantTables T;
    if constexpr (!BATCH) {
        // While the kernel before this one in the stream drains: ask L2 for this thread's first chunk.
        // A prefetch changes no architectural state and L2 is the point of coherence, so this is safe
        // even if that kernel is still writing x; the loads themselves come after the wait below.
        const size_t first = (size_t)blockIdx.x * kThreads + threadIdx.x;
        if (first < p.n_items)
            asm volatile("prefetch.global.L2 [%0];" ::"l"(static_cast<const char*>(p.x) + first * ((size_t)S::C * S::EB)));
    }
    wait_for_prior_grid();
    release_dependents();
    if constexpr (BATCH) {
        quantize_batch_body<DT, B, FMT, DUAL>(p, T, ring);
        return;
    }
    // request the first chunks before anything else: their latency hides behind the table build
    const size_t stride = (size_t)gridDim.x * kThreads;
    const int lane = threadIdx.x & 31;
    size_t chunk = (size_t)blockIdx.x * kThreads + threadIdx.x;
    const size_t wchunk0 = chunk - lane;   // chunk of the warp's lane 0
    constexpr size_t kChunkBytes = (size_t)S::C * S::EB;
    constexpr uint32_t kSlotBytes = S::PIECES * kThreads * 16;
    constexpr int DIST = S::SLOTS - 1;   // chunks requested ahead of the one being processed
    // first column of this warp in slot 0; a thread's own column is `lane` further
    const uint32_t ring_warp = (uint32_t)__cvta_generic_to_shared(ring) + (threadIdx.x - lane) * 16;
    const uint32_t ring_base = ring_warp + lane * 16;
    const char* x = static_cast<const char*>(p.x);
    {
        size_t c = S::COOP ? wchunk0 : chunk;
#pragma unroll
        for (int d = 0; d < DIST; ++d) {
            if constexpr (S::COOP) stage_warp_chunks<S::PIECES>(ring_warp + d * kSlotBytes, x, kChunkBytes, c, p.n_items, lane);
            else stage_chunk<S::PIECES>(ring_base + d * kSlotBytes, x + c * kChunkBytes, c < p.n_items);
            c += stride;
        }
    }
    QuantConsts k;
    k.g = p.d_global_scale ? *p.d_global_scale : p.global_scale;
    int first_bad;
    k.onemul = build_quant_tables<FMT, DT == kBF16>(T, k.g, first_bad);
    k.unit_g = (k.g == 1.0f);
    k.c_min = (p.prevent_zero && FMT != kUE8M0) ? 1 : 0;
    k.pow2_rule = (FMT == kUE8M0) ? p.pow2_rule : kPow2Eq1;
    k.u_floor = k.c_min ? __fmul_rn(4.0f, scale_value(FMT, 1)) : 0.0f;
    k.lean_cmax = first_bad - 1;
    k.Rg = 1.0f;
    // Ranges of a block maximum m for which u = fl(m / g) and fl(u / 6) come out exact from the
    // multiply-and-correct forms.  The FP8 formats round every u below 2^-20 to code 0, so an
    // inexact tiny quotient cannot change their code; the power-of-two format reads the exponent
    // of the quotient and needs it exact.
    k.need_lo = (FMT == kUE8M0) || !k.unit_g;
    k.m_hi = kFastMax;
    k.m_lo = 0.0f;
    if (k.unit_g) {
        if (FMT == kUE8M0) k.m_lo = 1.0e-30f;
    } else if (k.g >= kFastMin && k.g <= kFastMax) {
        k.Rg = __frcp_rn(k.g);
        k.m_hi = fminf(kFastMax, __fmul_rn(k.g, 1.0e29f));
        k.m_lo = fmaxf(1.084202172485504434e-19f /* 2^-63 */, (FMT == kUE8M0) ? __fmul_rn(k.g, 1.0e-29f) : 0.0f);
    } else {
        k.m_hi = -1.0f;   // tensor scale outside the shortcut range: general path everywhere
        k.m_lo = 0.0f;
    }

    // Thread-private staging: a thread leaves when its chunks are done (no barrier follows).
    // Cooperative staging: the warp stays together, lanes past the end only take part in the copies.
    // (with fused MSE partial sums every thread stays for the CTA-wide sum at the end)
    const bool has_work = (S::COOP ? wchunk0 : chunk) < p.n_items;
    if (!has_work && (FAKE || p.mse_partials == nullptr)) return;
    double sse_sum = 0.0;   // binary64 sum of the SSEs of this thread's blocks, in the order it produced them
    // The chunk loop, instantiated with and without the lean per-block path (see quantize_chunk);
    // which one runs is the same for every thread of the launch.
    auto chunk_loop = [&](auto lean_tag) {
        constexpr int LEAN = decltype(lean_tag)::value;
        int slot = 0;                      // slot holding `chunk`
        int fill = DIST % S::SLOTS;        // slot that the next request goes to
        size_t ahead = (S::COOP ? wchunk0 : chunk) + (size_t)DIST * stride;
        for (size_t lead = S::COOP ? wchunk0 : chunk; lead < p.n_items; lead += stride, chunk += stride) {
            // all but the DIST - 1 most recent groups are complete: this thread's copies for `chunk` have landed
            asm volatile("cp.async.wait_group %0;" ::"n"(DIST - 1) : "memory");
            // cooperative staging: so have the other lanes' copies, and every lane is done reading the
            // slot that the next request overwrites
            if constexpr (S::COOP) __syncwarp();
            const uint4* slot_warp = ring + (size_t)slot * (S::PIECES * kThreads) + (threadIdx.x - lane);
            // the slot read one trip ago is free again (its words were consumed by the arithmetic of
            // that trip): request the chunk DIST trips ahead into it.  The slot of the current chunk
            // is not requested into before the next trip, so it may be read throughout this one.
            if constexpr (S::COOP) stage_warp_chunks<S::PIECES>(ring_warp + fill * kSlotBytes, x, kChunkBytes, ahead, p.n_items, lane);
            else stage_chunk<S::PIECES>(ring_base + fill * kSlotBytes, x + ahead * kChunkBytes, ahead < p.n_items);
            ahead += stride;
            slot = (slot + 1 == S::SLOTS) ? 0 : slot + 1;
            fill = (fill + 1 == S::SLOTS) ? 0 : fill + 1;
            if (S::COOP && chunk >= p.n_items) continue;   // a lane past the end (the warp's last trip)
            // blocks longer than 16 elements go part by part, except 4-over-6 at B = 32, which measured
            // slightly faster with the whole block in registers
            if constexpr (long_block_path(B, DUAL)) {
                quantize_long_block<DT, B, FMT, DUAL, FAKE>(p, T, k, chunk, slot_warp, lane, sse_sum);
            } else {
                uint32_t raw[S::PIECES * 4];
#pragma unroll
                for (int q = 0; q < S::PIECES; ++q) {
                    const uint4 w = slot_warp[ring_index<S::COOP>(q, lane)];
                    raw[4 * q + 0] = w.x; raw[4 * q + 1] = w.y; raw[4 * q + 2] = w.z; raw[4 * q + 3] = w.w;
                }
                quantize_chunk<DT, B, FMT, DUAL, FAKE, LEAN>(p, T, k, chunk, raw, sse_sum);
            }
        }
    };
    constexpr bool CAN_LEAN = (DT == kBF16) && (FMT != kUE8M0) && !(long_block_path(B, DUAL));
    if (has_work) {
        if constexpr (CAN_LEAN) {
            if (lean_allowed<FMT>(first_bad, k.unit_g)) chunk_loop(std::integral_constant<int, 1>{});
            else if (lean_scaled_allowed(k)) chunk_loop(std::integral_constant<int, 2>{});
            else chunk_loop(std::integral_constant<int, 0>{});
        } else {
            chunk_loop(std::integral_constant<int, 0>{});
        }
    }
    if constexpr (!FAKE) {
        if (p.mse_partials != nullptr) {   // launch-uniform: every thread of the CTA is here
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            __syncthreads();               // the table is no longer read: its memory serves as scratch
            const double total = cta_sum_fixed_order(sse_sum, reinterpret_cast<double*>(&T));
            if (threadIdx.x == 0) p.mse_partials[p.mse_first + blockIdx.x] = total;
        }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
}

// Host side: pick the instantiation, launch a persistent grid over the whole chunks and hand the
// blocks past the last whole chunk to the scalar tail kernel.
template <int DT, int B, int FMT, bool DUAL, bool FAKE>
static cudaError_t launch_quantize_inst(const QuantArgs& a, cudaStream_t stream) {
    using S = QuantShape<DT, B>;
    static std::atomic<int> ctas_per_sm[kMaxDevices];   // first-use cache; racing threads store the same value
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    int resident = ctas_per_sm[dev].load(std::memory_order_relaxed);
    if (resident == 0) {
        err = cudaFuncSetAttribute(k_quantize<DT, B, FMT, DUAL, FAKE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   (int)S::RING_BYTES);
        if (err != cudaSuccess) return err;
        int n = 0;
        err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, k_quantize<DT, B, FMT, DUAL, FAKE>, kThreads, S::RING_BYTES);
        if (err != cudaSuccess) return err;
        resident = n > 0 ? n : 1;
        ctas_per_sm[dev].store(resident, std::memory_order_relaxed);
    }
    const size_t n_blocks = a.n_items;
    const size_t n_chunks = n_blocks / S::NBC;
    const size_t done = n_chunks * S::NBC;
    // The blocks past the last whole chunk go to the one-warp tail kernel.  With fused MSE partial sums it
    // runs first and owns partial 0; the CTAs of the main kernel own the partials from 1 on.
    auto launch_tail = [&]() -> cudaError_t {
        if (done == n_blocks) return cudaSuccess;
        QuantArgs t = a;
        t.first_item = done;
        t.n_items = n_blocks - done;
        t.mse_first = 0;
        return launch_quantize_tail(t, DT, B, FMT, DUAL, stream);
    };
    if (a.mse_partials) {
        err = launch_tail();
        if (err != cudaSuccess) return err;
    }
    if (n_chunks > 0) {
        QuantArgs m = a;
        m.n_items = n_chunks;
        m.mse_first = (done < n_blocks) ? 1 : 0;
        const size_t want = (n_chunks + kThreads - 1) / kThreads;
        size_t cap = (size_t)sm_count(dev) * (size_t)resident;
        if (a.mse_partials && cap > (size_t)kMsePartials - 1) cap = kMsePartials - 1;
        const unsigned grid = (unsigned)(want < cap ? want : cap);
        err = launch_pdl(k_quantize<DT, B, FMT, DUAL, FAKE>, grid, kThreads, S::RING_BYTES, stream, m);
        count_launch();
        if (err != cudaSuccess) return err;
        if (a.mse_n_partials) *a.mse_n_partials = (int)grid + m.mse_first;
    } else if (a.mse_n_partials) {
        *a.mse_n_partials = (done < n_blocks) ? 1 : 0;
    }
    if (!a.mse_partials) err = launch_tail();
    return err;
}

template <int DT, int B, int FMT, bool FAKE>
static cudaError_t launch_quantize_kind(const QuantArgs& a, bool dual, cudaStream_t s) {
    return dual ? launch_quantize_inst<DT, B, FMT, true, FAKE>(a, s) : launch_quantize_inst<DT, B, FMT, false, FAKE>(a, s);
}

template <int DT, int B, bool FAKE>
static cudaError_t launch_quantize_fmt(const QuantArgs& a, int fmt, bool dual, cudaStream_t s) {
    switch (fmt) {
    case kUE8M0: return launch_quantize_kind<DT, B, kUE8M0, FAKE>(a, dual, s);
    case kUE4M3: return launch_quantize_kind<DT, B, kUE4M3, FAKE>(a, dual, s);
    default: return launch_quantize_kind<DT, B, kUE5M3, FAKE>(a, dual, s);
    }
}

// FAKE = the fused fake-quantize variant (writes x_hat instead of codes, scales and SSE).
template <int DT, bool FAKE>
static cudaError_t launch_quantize_dt(const QuantArgs& a, int B, int fmt, bool dual, cudaStream_t s) {
    switch (B) {
    case 2: return launch_quantize_fmt<DT, 2, FAKE>(a, fmt, dual, s);
    case 4: return launch_quantize_fmt<DT, 4, FAKE>(a, fmt, dual, s);
    case 8: return launch_quantize_fmt<DT, 8, FAKE>(a, fmt, dual, s);
    case 16: return launch_quantize_fmt<DT, 16, FAKE>(a, fmt, dual, s);
    case 32: return launch_quantize_fmt<DT, 32, FAKE>(a, fmt, dual, s);
    default: return launch_quantize_fmt<DT, 64, FAKE>(a, fmt, dual, s);
    }
}

// Multi-tensor launch: one persistent grid over all rows of all tensors.
template <int DT, int B, int FMT, bool DUAL>
static cudaError_t launch_quantize_batch_inst(const QuantArgs& a, size_t total_rows, cudaStream_t stream) {
    using S = QuantShape<DT, B>;
    static std::atomic<int> ctas_per_sm[kMaxDevices];   // first-use cache; racing threads store the same value
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    int resident = ctas_per_sm[dev].load(std::memory_order_relaxed);
    if (resident == 0) {
        err = cudaFuncSetAttribute(k_quantize<DT, B, FMT, DUAL, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   (int)S::RING_BYTES);
        if (err != cudaSuccess) return err;
        int n = 0;
        err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, k_quantize<DT, B, FMT, DUAL, false, true>, kThreads, S::RING_BYTES);
        if (err != cudaSuccess) return err;
        resident = n > 0 ? n : 1;
        ctas_per_sm[dev].store(resident, std::memory_order_relaxed);
    }
    const size_t want = (total_rows + kThreads / 32 - 1) / (kThreads / 32);
    const size_t cap = (size_t)sm_count(dev) * (size_t)resident;
    const unsigned grid = (unsigned)(want < cap ? want : cap);
    err = launch_pdl(k_quantize<DT, B, FMT, DUAL, false, true>, grid, kThreads, S::RING_BYTES, stream, a);
    count_launch();
    return err;
}

template <int DT, int B>
static cudaError_t launch_quantize_batch_fmt(const QuantArgs& a, int fmt, bool dual, size_t rows, cudaStream_t s) {
    switch (fmt) {
    case kUE8M0: return dual ? launch_quantize_batch_inst<DT, B, kUE8M0, true>(a, rows, s) : launch_quantize_batch_inst<DT, B, kUE8M0, false>(a, rows, s);
    case kUE4M3: return dual ? launch_quantize_batch_inst<DT, B, kUE4M3, true>(a, rows, s) : launch_quantize_batch_inst<DT, B, kUE4M3, false>(a, rows, s);
    default: return dual ? launch_quantize_batch_inst<DT, B, kUE5M3, true>(a, rows, s) : launch_quantize_batch_inst<DT, B, kUE5M3, false>(a, rows, s);
    }
}

template <int DT>
static cudaError_t launch_quantize_batch_dt(const QuantArgs& a, int B, int fmt, bool dual, size_t rows, cudaStream_t s) {
    switch (B) {
    case 2: return launch_quantize_batch_fmt<DT, 2>(a, fmt, dual, rows, s);
    case 4: return launch_quantize_batch_fmt<DT, 4>(a, fmt, dual, rows, s);
    case 8: return launch_quantize_batch_fmt<DT, 8>(a, fmt, dual, rows, s);
    case 16: return launch_quantize_batch_fmt<DT, 16>(a, fmt, dual, rows, s);
    case 32: return launch_quantize_batch_fmt<DT, 32>(a, fmt, dual, rows, s);
    default: return launch_quantize_batch_fmt<DT, 64>(a, fmt, dual, rows, s);
    }
}

}  // namespace mxq
