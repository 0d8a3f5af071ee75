// Fused one-pass quantization kernels: block amax -> scale code -> FP4 codes -> block SSE.
//   kind SINGLE  abs-max (Eq. 2; Eq. 1 for UE8M0), optional prevent-zero clamp (Eq. 3)
//   kind DUAL    4-over-6 (Eq. 4): candidates for M = 6 and M = 4, keep the smaller SSE
// One thread owns a chunk of C = max(B, 8) consecutive elements (one block, or 8/B small
// blocks), so every per-block quantity lives in registers and the SSE is accumulated in element
// order.  CTAs are persistent (grid = SMs x resident CTAs) and build the per-code decode-scale
// tables once in shared memory.
#pragma once

#include "mxq_device.cuh"
#include "mxq_internal.h"

namespace mxq {

template <int B, int N>
__device__ __forceinline__ void block_amax(const float (&v)[N], float (&a)[N / B]) {
#pragma unroll
    for (int j = 0; j < N / B; ++j) {
        float m = 0.0f;
#pragma unroll
        for (int i = 0; i < B; ++i) m = fmaxf(m, fabsf(v[j * B + i]));
        a[j] = m;
    }
}

// Quantize the C elements of a chunk with one scale code per block; returns packed codes and
// per-block SSE (e = fma(-q, D, v); sse = fma(e, e, sse), in element order).
template <int B, int C>
__device__ __forceinline__ void encode_chunk(const float (&v)[C], const float (&amax)[C / B], const int (&code)[C / B],
                                             const float* tabD, const float* tabR, uint32_t (&packed)[C / 8],
                                             float (&sse)[C / B]) {
    constexpr int NB = C / B;
    float t[C];
    float D[NB];
#pragma unroll
    for (int j = 0; j < NB; ++j) {
        D[j] = tabD[code[j]];
        const float R = tabR[code[j]];
        if (R != 0.0f && amax[j] <= kFastMax) {
#pragma unroll
            for (int i = 0; i < B; ++i) t[j * B + i] = quotient_corrected(v[j * B + i], D[j], R);
        } else {
#pragma unroll
            for (int i = 0; i < B; ++i) t[j * B + i] = quotient_general(v[j * B + i], D[j]);
        }
    }
    float q[C];
#pragma unroll
    for (int k = 0; k < C / 8; ++k) {
        float q8[8];
        packed[k] = quantize_e2m1x8(&t[8 * k], q8);
#pragma unroll
        for (int i = 0; i < 8; ++i) q[8 * k + i] = q8[i];
    }
#pragma unroll
    for (int j = 0; j < NB; ++j) {
        float s = 0.0f;
#pragma unroll
        for (int i = 0; i < B; ++i) {
            const float e = __fmaf_rn(-q[j * B + i], D[j], v[j * B + i]);
            s = __fmaf_rn(e, e, s);
        }
        sse[j] = s;
    }
}

template <int DT, int B, int FMT, bool DUAL>
__global__ void __launch_bounds__(kThreads) k_quantize(QuantArgs p) {
    constexpr int C = (B < 8) ? 8 : B;
    constexpr int NB = C / B;
    __shared__ float tabD[256];
    __shared__ float tabR[256];
    const float g = p.d_global_scale ? *p.d_global_scale : p.global_scale;
    build_scale_tables<FMT>(tabD, tabR, g);
    const bool unit_g = (g == 1.0f);
    const bool pz = p.prevent_zero && FMT != kUE8M0;

    const size_t stride = (size_t)gridDim.x * kThreads;
    for (size_t chunk = (size_t)blockIdx.x * kThreads + threadIdx.x; chunk < p.n_items; chunk += stride) {
        float v[C];
        load_elems<DT, C>(p.x, chunk * C, v);
        float amax[NB];
        block_amax<B, C>(v, amax);

        int c6[NB];
        float u[NB];
#pragma unroll
        for (int j = 0; j < NB; ++j) {
            u[j] = unit_g ? amax[j] : __fdiv_rn(amax[j], g);
            c6[j] = round_scale<FMT>(__fdiv_rn(u[j], 6.0f));
            if (pz) c6[j] = max(c6[j], 1);
        }
        uint32_t packed[C / 8];
        float sse[NB];
        encode_chunk<B, C>(v, amax, c6, tabD, tabR, packed, sse);

        if constexpr (DUAL) {
            int c4[NB];
            bool any = false;
#pragma unroll
            for (int j = 0; j < NB; ++j) {
                c4[j] = round_scale<FMT>(__fdiv_rn(u[j], 4.0f));
                if (pz) c4[j] = max(c4[j], 1);
                any |= (c4[j] != c6[j]);
            }
            if (any) {
                uint32_t packed4[C / 8];
                float sse4[NB];
                encode_chunk<B, C>(v, amax, c4, tabD, tabR, packed4, sse4);
                if constexpr (NB == 1) {
                    if (sse4[0] < sse[0]) {
                        sse[0] = sse4[0];
                        c6[0] = c4[0];
#pragma unroll
                        for (int k = 0; k < C / 8; ++k) packed[k] = packed4[k];
                    }
                } else {
                    // several blocks share the one 32-bit code word: select by bit mask
                    constexpr uint32_t kBlockMask = (B == 2) ? 0xFFu : 0xFFFFu;
                    uint32_t take = 0;
#pragma unroll
                    for (int j = 0; j < NB; ++j) {
                        if (sse4[j] < sse[j]) {
                            sse[j] = sse4[j];
                            c6[j] = c4[j];
                            take |= kBlockMask << (j * 4 * B);
                        }
                    }
                    packed[0] = (packed4[0] & take) | (packed[0] & ~take);
                }
            }
        }

        store_bytes<C / 2>(p.codes + chunk * (C / 2), packed);
        uint32_t sc = 0;
#pragma unroll
        for (int j = 0; j < NB; ++j) sc |= (uint32_t)c6[j] << (8 * j);
        store_bytes<NB>(p.scales + chunk * NB, &sc);
        if (p.block_sse) {
            uint32_t sw[NB];
#pragma unroll
            for (int j = 0; j < NB; ++j) sw[j] = __float_as_uint(sse[j]);
            store_bytes<4 * NB>(p.block_sse + chunk * NB, sw);
        }
    }
}

// Host side: pick the instantiation and launch a persistent grid.
template <int DT, int B, int FMT, bool DUAL>
static cudaError_t launch_quantize_inst(const QuantArgs& a, cudaStream_t stream) {
    static int ctas_per_sm[kMaxDevices] = {0};
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    if (ctas_per_sm[dev] == 0) {
        int n = 0;
        err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, k_quantize<DT, B, FMT, DUAL>, kThreads, 0);
        if (err != cudaSuccess) return err;
        ctas_per_sm[dev] = n > 0 ? n : 1;
    }
    const size_t want = (a.n_items + kThreads - 1) / kThreads;
    const size_t cap = (size_t)sm_count(dev) * (size_t)ctas_per_sm[dev];
    const unsigned grid = (unsigned)(want < cap ? want : cap);
    k_quantize<DT, B, FMT, DUAL><<<grid, kThreads, 0, stream>>>(a);
    count_launch();
    return cudaGetLastError();
}

template <int DT, int B, int FMT>
static cudaError_t launch_quantize_kind(const QuantArgs& a, bool dual, cudaStream_t s) {
    return dual ? launch_quantize_inst<DT, B, FMT, true>(a, s) : launch_quantize_inst<DT, B, FMT, false>(a, s);
}

template <int DT, int B>
static cudaError_t launch_quantize_fmt(const QuantArgs& a, int fmt, bool dual, cudaStream_t s) {
    switch (fmt) {
    case kUE8M0: return launch_quantize_kind<DT, B, kUE8M0>(a, dual, s);
    case kUE4M3: return launch_quantize_kind<DT, B, kUE4M3>(a, dual, s);
    default: return launch_quantize_kind<DT, B, kUE5M3>(a, dual, s);
    }
}

template <int DT>
static cudaError_t launch_quantize_dt(const QuantArgs& a, int B, int fmt, bool dual, cudaStream_t s) {
    switch (B) {
    case 2: return launch_quantize_fmt<DT, 2>(a, fmt, dual, s);
    case 4: return launch_quantize_fmt<DT, 4>(a, fmt, dual, s);
    case 8: return launch_quantize_fmt<DT, 8>(a, fmt, dual, s);
    case 16: return launch_quantize_fmt<DT, 16>(a, fmt, dual, s);
    case 32: return launch_quantize_fmt<DT, 32>(a, fmt, dual, s);
    default: return launch_quantize_fmt<DT, 64>(a, fmt, dual, s);
    }
}

}  // namespace mxq
