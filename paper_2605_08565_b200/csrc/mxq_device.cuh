// Device-side building blocks of libmxq (sm_100a): scale-format tables, scale rounding, FP4
// conversion wrappers and the exact per-element quotient.  Every floating-point step uses an
// explicit round-to-nearest intrinsic so that the compiler can neither contract nor reorder it.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "mxq_internal.h"

namespace mxq {

constexpr int kF32 = 0, kBF16 = 1;
constexpr int kUE8M0 = 0, kUE4M3 = 1, kUE5M3 = 2;
constexpr int kThreads = 256;

// See launch_pdl(): holds a programmatically staged grid until the kernel before it in the stream
// has completed and its writes are visible.
__device__ __forceinline__ void wait_for_prior_grid() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Lets the next kernel of the stream (if it was launched with programmatic stream serialization) be
// staged onto SM resources as they become free, so that its launch latency and prologue overlap
// this kernel's tail.  It still blocks in its own wait_for_prior_grid() until this grid has
// completed and flushed its writes, so the ordering of a plain stream is kept.  The dependent grid
// is released only after EVERY CTA of this grid has executed this instruction (or exited), i.e.
// when all of them are resident or done: the staged CTAs can never keep this grid off the SMs.
__device__ __forceinline__ void release_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Sum of one binary64 value per thread over a CTA of kThreads threads, in a fixed order (a shuffle
// tree inside each warp, then the warps in order): the same inputs give the same bits.  Every
// thread of the CTA must call it; the result is valid in thread 0.  scratch: kThreads / 32 doubles
// of shared memory that nothing else uses until the next barrier.
__device__ __forceinline__ double cta_sum_fixed_order(double v, double* scratch) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = __dadd_rn(v, __shfl_down_sync(0xFFFFFFFFu, v, o));
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    double t = 0.0;
    if (threadIdx.x == 0) {
#pragma unroll
        for (int w = 0; w < kThreads / 32; ++w) t = __dadd_rn(t, scratch[w]);
    }
    return t;
}

// Tail kernels (one warp): the binary64 sum of one SSE per lane, shuffle tree in fixed order, stored
// as the call's partial number p.mse_first.  Every lane of the warp calls it (0 for an idle lane).
__device__ __forceinline__ void warp_sum_to_partial(const QuantArgs& p, float sse) {
    double v = (double)sse;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = __dadd_rn(v, __shfl_down_sync(0xFFFFFFFFu, v, o));
    if ((threadIdx.x & 31) == 0) p.mse_partials[p.mse_first] = v;
}

__host__ __device__ constexpr int num_codes(int fmt) { return fmt == kUE4M3 ? 127 : 255; }
__host__ __device__ constexpr int elem_bytes(int dt) { return dt == kF32 ? 4 : 2; }

// Largest magnitude for which the multiply-and-correct quotient below is used.
constexpr float kFastMax = 1.152921504606846976e18f;   // 2^60
constexpr float kFastMin = 8.673617379884035472e-19f;  // 2^-60

// Decoded value of a block-scale code (Background: E8M0 powers of two; E4M3 with the sign bit
// unused, smallest nonzero 2^-9; UE5M3 taken as bias 15 with subnormals).
__device__ __forceinline__ float scale_value(int fmt, int c) {
    if (fmt == kUE8M0) return __uint_as_float(c == 0 ? 0x00400000u : (uint32_t)c << 23);
    const int bias = (fmt == kUE4M3) ? 7 : 15;
    const int e = c >> 3, m = c & 7;
    if (e == 0) return __fmul_rn(__int2float_rn(m), __uint_as_float((uint32_t)(127 - bias - 2) << 23));
    return __uint_as_float(((uint32_t)(e - bias + 127) << 23) | ((uint32_t)m << 20));
}

// Round_SF of Eq. 2 (round-to-nearest-even onto the format, clipped to the largest finite code)
// and the floor rule of Eq. 1 for the power-of-two format.  w >= 0.
template <int FMT>
__device__ __forceinline__ int round_scale(float w) {
    if constexpr (FMT == kUE8M0) {
        // 2^(c-127) <= w < 2^(c-126): c is the biased exponent field; denormals give 0.
        return (int)min(__float_as_uint(w) >> 23, 254u);
    } else if constexpr (FMT == kUE4M3) {
        uint16_t r;
        asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(0.0f), "f"(w));
        return r & 0xFF;
    } else {
        const uint32_t b = __float_as_uint(w);
        if (b >= 0x47E00000u) return 0xFE;                                            // >= 1.75 * 2^16
        if (b < 0x38800000u) return __float2int_rn(__fmul_rn(w, 131072.0f));           // < 2^-14: m * 2^-17
        uint32_t r = b - 0x38000000u;                                                  // rebias 127 -> 15
        r += 0x7FFFFu + ((r >> 20) & 1u);                                              // RNE to 3 mantissa bits
        return (int)(r >> 20);
    }
}

// The OCP MX wording of the power-of-two rule: scale exponent = exponent of the (tensor-scale
// adjusted) block maximum minus the exponent of the largest FP4 value (2), clamped to the codes.
__device__ __forceinline__ int ocp_scale_code(float u) {
    const uint32_t b = __float_as_uint(u);               // u >= 0; subnormal u has exponent field 0
    if (b >= 0x7F800000u) return 254;                    // amax / g overflowed: the largest scale
    return max((int)(b >> 23) - 2, 0);
}

// The power-of-two scale that maps the (tensor-scale adjusted) block maximum u into [3.5, 7):
// exponent floor(log2(u / 3.5)).  With u = m * 2^E, 1 <= m < 2, u / 3.5 = (m / 1.75) * 2^(E - 1),
// so the exponent is E - 2 when m < 1.75 and E - 1 otherwise.
__device__ __forceinline__ int clip7_scale_code(float u) {
    const uint32_t b = __float_as_uint(u);
    if (b >= 0x7F800000u) return 254;
    return max((int)(b >> 23) - 2 + ((b & 0x007FFFFFu) >= 0x00600000u ? 1 : 0), 0);
}

// Scale code of the alternative power-of-two rules (rule != kPow2Eq1).
__device__ __forceinline__ int pow2_rule_code(float u, int rule) {
    return rule == kPow2Ocp ? ocp_scale_code(u) : clip7_scale_code(u);
}

// Per-CTA lookup tables: D[c] = fl32(value(c) * g) and R[c] = RN(1 / D[c]), or R[c] = 0 when the
// multiply-and-correct quotient must not be used with this scale (D zero, tiny, huge or not finite).
template <int FMT>
__device__ __forceinline__ void build_scale_tables(float* tabD, float* tabR, float g) {
    for (int c = threadIdx.x; c < 256; c += blockDim.x) {
        float D = __uint_as_float(0x7FC00000u), R = 0.0f;
        if (c < num_codes(FMT)) {
            D = __fmul_rn(scale_value(FMT, c), g);
            if (D >= kFastMin && D <= kFastMax) R = __frcp_rn(D);
        }
        tabD[c] = D;
        tabR[c] = R;
    }
    __syncthreads();
}

// fl32(v / D) for kFastMin <= D <= kFastMax, |v| <= kFastMax, R = RN(1/D): a reciprocal multiply
// followed by one residual correction, which is the IEEE quotient for every such pair (the
// argument and the enumeration of the hard cases are with quotient_short() of the one-pass
// kernels; magnitudes below 2^-62 may lose the residual to underflow, but their quotients stay far
// below the first FP4 decision point, 0.25, or they are sent to the general path).  The residual is
// formed as (q*D - v) so that a zero quotient keeps the sign of v.
__device__ __forceinline__ float quotient_corrected(float v, float D, float R) {
    const float q = __fmul_rn(v, R);
    const float r = __fmaf_rn(q, D, -v);
    return __fmaf_rn(-r, R, q);
}

// General quotient: IEEE division; a zero scale sends every element to (signed) zero.
__device__ __forceinline__ float quotient_general(float v, float D) {
    return (D == 0.0f) ? __fmul_rn(v, 0.0f) : __fdiv_rn(v, D);
}

// Eight quotients -> eight FP4 codes in one word (element 0 in bits 0..3): round-to-nearest-even
// onto the E2M1 grid with saturation at +-6; the sign bit of a zero result is kept.
__device__ __forceinline__ uint32_t pack_e2m1x8(float t0, float t1, float t2, float t3, float t4, float t5,
                                                float t6, float t7) {
    uint32_t out;
    asm("{\n"
        " .reg .b8 b0, b1, b2, b3;\n"
        " cvt.rn.satfinite.e2m1x2.f32 b0, %2, %1;\n"
        " cvt.rn.satfinite.e2m1x2.f32 b1, %4, %3;\n"
        " cvt.rn.satfinite.e2m1x2.f32 b2, %6, %5;\n"
        " cvt.rn.satfinite.e2m1x2.f32 b3, %8, %7;\n"
        " mov.b32 %0, {b0, b1, b2, b3};\n"
        "}"
        : "=r"(out)
        : "f"(t0), "f"(t1), "f"(t2), "f"(t3), "f"(t4), "f"(t5), "f"(t6), "f"(t7));
    return out;
}

// Two quotients -> one byte of two FP4 codes (in bits 0..7 of the result).
__device__ __forceinline__ uint32_t pack_e2m1x2(float t0, float t1) {
    uint32_t out;
    asm("{\n"
        " .reg .b8 b0;\n"
        " .reg .b16 h;\n"
        " cvt.rn.satfinite.e2m1x2.f32 b0, %2, %1;\n"
        " mov.b16 h, {b0, b0};\n"
        " cvt.u32.u16 %0, h;\n"
        "}"
        : "=r"(out)
        : "f"(t0), "f"(t1));
    return out & 0xFFu;
}

// Eight FP4 codes -> eight floats (exact).  Each byte is split off with integer shifts and handed
// to the converter through a 16-bit register pair.
__device__ __forceinline__ void unpack_e2m1x8(uint32_t codes, float (&q)[8]) {
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        uint32_t h;
        const uint16_t b = (uint16_t)((codes >> (8 * k)) & 0xFFu);
        asm("{\n"
            " .reg .b8 lo, hi;\n"
            " mov.b16 {lo, hi}, %1;\n"
            " cvt.rn.f16x2.e2m1x2 %0, lo;\n"
            "}"
            : "=r"(h)
            : "h"(b));
        const float2 f = __half22float2(*reinterpret_cast<__half2*>(&h));
        q[2 * k] = f.x;
        q[2 * k + 1] = f.y;
    }
}

// Two quotients -> the two grid values they round to, as floats (no code kept).
__device__ __forceinline__ float2 round_e2m1x2(float t0, float t1) {
    uint32_t h;
    asm("{\n"
        " .reg .b8 b0;\n"
        " cvt.rn.satfinite.e2m1x2.f32 b0, %2, %1;\n"
        " cvt.rn.f16x2.e2m1x2 %0, b0;\n"
        "}"
        : "=r"(h)
        : "f"(t0), "f"(t1));
    return __half22float2(*reinterpret_cast<__half2*>(&h));
}

// Read BYTES consecutive bytes (BYTES = 4, 8 or a multiple of 16; pointer aligned to
// min(BYTES, 16)) with streaming loads and widen to floats.
template <int DT, int N>
__device__ __forceinline__ void load_elems(const void* base, size_t first_elem, float (&v)[N]) {
    constexpr int BYTES = N * elem_bytes(DT);
    constexpr int WORDS = BYTES / 4;
    uint32_t w[WORDS];
    const char* p = static_cast<const char*>(base) + first_elem * (size_t)elem_bytes(DT);
    if constexpr (BYTES == 4) {
        w[0] = __ldcs(reinterpret_cast<const uint32_t*>(p));
    } else if constexpr (BYTES == 8) {
        const uint2 t = __ldcs(reinterpret_cast<const uint2*>(p));
        w[0] = t.x; w[1] = t.y;
    } else {
        static_assert(BYTES % 16 == 0, "unsupported chunk size");
#pragma unroll
        for (int k = 0; k < BYTES / 16; ++k) {
            const uint4 t = __ldcs(reinterpret_cast<const uint4*>(p) + k);
            w[4 * k + 0] = t.x; w[4 * k + 1] = t.y; w[4 * k + 2] = t.z; w[4 * k + 3] = t.w;
        }
    }
    if constexpr (DT == kF32) {
#pragma unroll
        for (int i = 0; i < N; ++i) v[i] = __uint_as_float(w[i]);
    } else {
#pragma unroll
        for (int i = 0; i < N / 2; ++i) {
            v[2 * i + 0] = __uint_as_float(w[i] << 16);
            v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
}

// Write BYTES bytes held in 32-bit words (BYTES = 1, 2, 4, 8 or a multiple of 16).
template <int BYTES>
__device__ __forceinline__ void store_bytes(void* dst, const uint32_t* w) {
    if constexpr (BYTES == 1) {
        *static_cast<uint8_t*>(dst) = (uint8_t)w[0];
    } else if constexpr (BYTES == 2) {
        *static_cast<uint16_t*>(dst) = (uint16_t)w[0];
    } else if constexpr (BYTES == 4) {
        __stcs(static_cast<uint32_t*>(dst), w[0]);
    } else if constexpr (BYTES == 8) {
        __stcs(static_cast<uint2*>(dst), make_uint2(w[0], w[1]));
    } else {
        static_assert(BYTES % 16 == 0, "unsupported store size");
#pragma unroll
        for (int k = 0; k < BYTES / 16; ++k)
            __stcs(static_cast<uint4*>(dst) + k, make_uint4(w[4 * k], w[4 * k + 1], w[4 * k + 2], w[4 * k + 3]));
    }
}

}  // namespace mxq
