// Brute-force scale search (Experimental Setup: "a brute-force search over possible scaling
// factors to minimize the MSE"): every finite scale code of the format is tried on every block and
// the code with the smallest SSE is kept (equal SSE: the smaller code).
//
// One thread owns one block of B elements in registers.  The candidate loop is uniform across the
// CTA, so the candidate's decode scale D and its reciprocal come from the shared-memory tables as
// broadcast reads.  Per candidate and element: exact quotient, round onto the FP4 grid, residual
// FMA, square-accumulate FMA -- in element order, so the SSE has the same bits as in the one-pass
// kernels and in the final encode.
#pragma once

#include "mxq_device.cuh"
#include "mxq_internal.h"

namespace mxq {

template <int B, bool FAST>
__device__ __forceinline__ float candidate_sse(const float (&v)[B], float D, float R) {
    float s = 0.0f;
#pragma unroll
    for (int i = 0; i < B; i += 2) {
        float t0, t1;
        if constexpr (FAST) {
            t0 = quotient_corrected(v[i], D, R);
            t1 = quotient_corrected(v[i + 1], D, R);
        } else {
            t0 = quotient_general(v[i], D);
            t1 = quotient_general(v[i + 1], D);
        }
        const float2 q = round_e2m1x2(t0, t1);
        const float e0 = __fmaf_rn(-q.x, D, v[i]);
        s = __fmaf_rn(e0, e0, s);
        const float e1 = __fmaf_rn(-q.y, D, v[i + 1]);
        s = __fmaf_rn(e1, e1, s);
    }
    return s;
}

template <int DT, int B, int FMT>
__global__ void __launch_bounds__(kThreads) k_brute(QuantArgs p) {
    __shared__ float tabD[256];
    __shared__ float tabR[256];
    const float g = p.d_global_scale ? *p.d_global_scale : p.global_scale;
    build_scale_tables<FMT>(tabD, tabR, g);
    const int first = (p.prevent_zero && FMT != kUE8M0) ? 1 : 0;

    const size_t stride = (size_t)gridDim.x * kThreads;
    for (size_t blk = (size_t)blockIdx.x * kThreads + threadIdx.x; blk < p.n_items; blk += stride) {
        float v[B];
        load_elems<DT, B>(p.x, blk * B, v);
        float amax = 0.0f;
#pragma unroll
        for (int i = 0; i < B; ++i) amax = fmaxf(amax, fabsf(v[i]));
        const bool fast_ok = amax <= kFastMax;

        uint32_t best_bits = 0xFFFFFFFFu;
        int best = first;
        for (int c = first; c < num_codes(FMT); ++c) {
            const float D = tabD[c];
            const float R = tabR[c];
            if (!(fabsf(D) <= 3.402823466e38f)) continue;  // decode scale overflowed: not usable
            float s;
            if (R != 0.0f && fast_ok) s = candidate_sse<B, true>(v, D, R);
            else s = candidate_sse<B, false>(v, D, R);
            const uint32_t bits = __float_as_uint(s);  // s >= 0: integer order equals float order
            if (bits < best_bits) {
                best_bits = bits;
                best = c;
            }
        }

        // final encode with the winner
        const float D = tabD[best];
        const float R = tabR[best];
        const bool fast = (R != 0.0f) && fast_ok;
        float t[B];
#pragma unroll
        for (int i = 0; i < B; ++i) t[i] = fast ? quotient_corrected(v[i], D, R) : quotient_general(v[i], D);
        if constexpr (B >= 8) {
            uint32_t packed[B / 8];
#pragma unroll
            for (int k = 0; k < B / 8; ++k)
                packed[k] = pack_e2m1x8(t[8 * k], t[8 * k + 1], t[8 * k + 2], t[8 * k + 3], t[8 * k + 4],
                                        t[8 * k + 5], t[8 * k + 6], t[8 * k + 7]);
            store_bytes<B / 2>(p.codes + blk * (B / 2), packed);
        } else {
            uint32_t packed = 0;
#pragma unroll
            for (int k = 0; k < B / 2; ++k) packed |= pack_e2m1x2(t[2 * k], t[2 * k + 1]) << (8 * k);
            store_bytes<B / 2>(p.codes + blk * (B / 2), &packed);
        }
        p.scales[blk] = (uint8_t)best;
        if (p.block_sse) p.block_sse[blk] = __uint_as_float(best_bits);
    }
}

template <int DT, int B, int FMT>
static cudaError_t launch_brute_inst(const QuantArgs& a, cudaStream_t stream) {
    static int ctas_per_sm[kMaxDevices] = {0};
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    if (ctas_per_sm[dev] == 0) {
        int n = 0;
        err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, k_brute<DT, B, FMT>, kThreads, 0);
        if (err != cudaSuccess) return err;
        ctas_per_sm[dev] = n > 0 ? n : 1;
    }
    const size_t want = (a.n_items + kThreads - 1) / kThreads;
    const size_t cap = (size_t)sm_count(dev) * (size_t)ctas_per_sm[dev];
    const unsigned grid = (unsigned)(want < cap ? want : cap);
    k_brute<DT, B, FMT><<<grid, kThreads, 0, stream>>>(a);
    count_launch();
    return cudaGetLastError();
}

template <int DT, int B>
static cudaError_t launch_brute_fmt(const QuantArgs& a, int fmt, cudaStream_t s) {
    switch (fmt) {
    case kUE8M0: return launch_brute_inst<DT, B, kUE8M0>(a, s);
    case kUE4M3: return launch_brute_inst<DT, B, kUE4M3>(a, s);
    default: return launch_brute_inst<DT, B, kUE5M3>(a, s);
    }
}

template <int DT>
static cudaError_t launch_brute_dt(const QuantArgs& a, int B, int fmt, cudaStream_t s) {
    switch (B) {
    case 2: return launch_brute_fmt<DT, 2>(a, fmt, s);
    case 4: return launch_brute_fmt<DT, 4>(a, fmt, s);
    case 8: return launch_brute_fmt<DT, 8>(a, fmt, s);
    case 16: return launch_brute_fmt<DT, 16>(a, fmt, s);
    case 32: return launch_brute_fmt<DT, 32>(a, fmt, s);
    default: return launch_brute_fmt<DT, 64>(a, fmt, s);
    }
}

}  // namespace mxq
