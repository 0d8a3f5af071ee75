// Analysis kernels around the quantizer (Results, numerical study; Appendix: clipping-only MSE,
// entry and scale histograms): the clipping part of the block SSE, histograms of the FP4 codes and
// of the scale codes, and the MSE of equal-length segments of a tensor (one sigma of the
// numerical study per segment).  None of them is on the bandwidth-critical path; they are written
// for exactness and determinism first.
#include "mxq_device.cuh"
#include "mxq_internal.h"

namespace mxq {

// ------------------------------------------------------------------------------------------------
// Clipping part of the block SSE: elements with |fl32(v / D)| > 6 are all mapped to +-6; their
// error is accumulated exactly like the block SSE (e = fma(-q, D, v); s = fma(e, e, s), element
// order), the other elements are skipped.  A zero decode scale clips nothing.  One thread per
// block; IEEE division throughout.
// ------------------------------------------------------------------------------------------------
template <int DT, int B>
__global__ void __launch_bounds__(kThreads) k_block_clip_sse(const void* x, size_t n_blocks, int fmt, float g,
                                                             const float* d_g, const uint8_t* scales, float* out) {
    wait_for_prior_grid();
    release_dependents();
    const float gs = d_g ? *d_g : g;
    const size_t stride = (size_t)gridDim.x * kThreads;
    for (size_t b = (size_t)blockIdx.x * kThreads + threadIdx.x; b < n_blocks; b += stride) {
        float v[B];
        load_elems<DT, B>(x, b * B, v);      // vector loads: a block is 4 .. 256 contiguous bytes
        const int c = scales[b];
        float s = 0.0f;
        if (c < num_codes(fmt)) {
            const float D = __fmul_rn(scale_value(fmt, c), gs);
            if (D != 0.0f) {
#pragma unroll
                for (int i = 0; i < B; ++i) {
                    const float t = __fdiv_rn(v[i], D);
                    if (fabsf(t) > 6.0f) {
                        const float q = copysignf(6.0f, v[i]);
                        const float e = __fmaf_rn(-q, D, v[i]);
                        s = __fmaf_rn(e, e, s);
                    }
                }
            }
        } else {
            s = __uint_as_float(0x7FC00000u);   // not a code of the format
        }
        out[b] = s;
    }
}

template <int DT>
static cudaError_t launch_clip_dt(const void* x, size_t n_blocks, int B, int fmt, float g, const float* d_g,
                                  const uint8_t* scales, float* out, unsigned grid, cudaStream_t s) {
    switch (B) {
    case 2: return launch_pdl(k_block_clip_sse<DT, 2>, grid, kThreads, 0, s, x, n_blocks, fmt, g, d_g, scales, out);
    case 4: return launch_pdl(k_block_clip_sse<DT, 4>, grid, kThreads, 0, s, x, n_blocks, fmt, g, d_g, scales, out);
    case 8: return launch_pdl(k_block_clip_sse<DT, 8>, grid, kThreads, 0, s, x, n_blocks, fmt, g, d_g, scales, out);
    case 16: return launch_pdl(k_block_clip_sse<DT, 16>, grid, kThreads, 0, s, x, n_blocks, fmt, g, d_g, scales, out);
    case 32: return launch_pdl(k_block_clip_sse<DT, 32>, grid, kThreads, 0, s, x, n_blocks, fmt, g, d_g, scales, out);
    default: return launch_pdl(k_block_clip_sse<DT, 64>, grid, kThreads, 0, s, x, n_blocks, fmt, g, d_g, scales, out);
    }
}

cudaError_t launch_block_clip_sse(const void* x, int dtype, size_t n, int B, int fmt, float g, const float* d_g,
                                  const uint8_t* scales, float* out, cudaStream_t s) {
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    const size_t n_blocks = n / (size_t)B;
    size_t want = (n_blocks + kThreads - 1) / kThreads;
    const size_t cap = (size_t)sm_count(dev) * 8;
    const unsigned grid = (unsigned)(want < cap ? want : cap);
    err = (dtype == kF32) ? launch_clip_dt<kF32>(x, n_blocks, B, fmt, g, d_g, scales, out, grid, s)
                          : launch_clip_dt<kBF16>(x, n_blocks, B, fmt, g, d_g, scales, out, grid, s);
    count_launch();
    return err;
}

// ------------------------------------------------------------------------------------------------
// Histograms: 16 bins of the 4-bit codes, 256 bins of the scale codes, ADDED to the caller's
// 64-bit counters.  The pass is a byte histogram: a code byte holds two codes, so the kernel counts
// the 256 byte values (one shared-memory integer atomic per TWO codes, one private copy of the
// table per warp so that only lanes of one warp can collide) and folds them into the 16 code bins at
// the end; scale bytes are counted the same way.  16-byte loads, no per-code compares.  Per-CTA
// counts are 32-bit (a CTA sees far fewer than 2^32 bytes), flushed with 64-bit integer atomics --
// integer sums are order-free, so the result is deterministic.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ void count_bytes_of_word(unsigned int* tab, uint32_t w) {
    atomicAdd(tab + (w & 0xFFu), 1u);
    atomicAdd(tab + ((w >> 8) & 0xFFu), 1u);
    atomicAdd(tab + ((w >> 16) & 0xFFu), 1u);
    atomicAdd(tab + (w >> 24), 1u);
}

// Adds the byte histogram of p[0 .. n_bytes) to this warp's table: bytes up to the first 16-byte
// boundary and past the last one singly (by the first threads of the grid), the rest as 16-byte loads.
__device__ __forceinline__ void count_byte_range(unsigned int* tab, const uint8_t* p, size_t n_bytes, size_t tid, size_t stride) {
    size_t head = (16u - (size_t)(reinterpret_cast<uintptr_t>(p) & 15u)) & 15u;
    if (head > n_bytes) head = n_bytes;
    const size_t n_vec = (n_bytes - head) / 16;
    const size_t tail0 = head + n_vec * 16;
    const uint4* v = reinterpret_cast<const uint4*>(p + head);
    for (size_t i = tid; i < n_vec; i += stride) {
        const uint4 w = __ldcs(v + i);
        count_bytes_of_word(tab, w.x);
        count_bytes_of_word(tab, w.y);
        count_bytes_of_word(tab, w.z);
        count_bytes_of_word(tab, w.w);
    }
    if (tid < head) atomicAdd(tab + p[tid], 1u);
    if (tid < n_bytes - tail0) atomicAdd(tab + p[tail0 + tid], 1u);
}

__global__ void __launch_bounds__(kThreads) k_histograms(const uint8_t* codes, const uint8_t* scales, size_t n,
                                                         size_t n_blocks, unsigned long long* code_hist,
                                                         unsigned long long* scale_hist) {
    constexpr int kWarps = kThreads / 32;
    __shared__ unsigned int sh_byte[kWarps][256];    // code bytes (two codes each), one table per warp
    __shared__ unsigned int sh_scale[kWarps][256];
    __shared__ unsigned long long sh_code[16];
    for (int i = threadIdx.x; i < kWarps * 256; i += kThreads) {
        (&sh_byte[0][0])[i] = 0;
        (&sh_scale[0][0])[i] = 0;
    }
    if (threadIdx.x < 16) sh_code[threadIdx.x] = 0;
    __syncthreads();
    const size_t stride = (size_t)gridDim.x * kThreads;
    const size_t tid = (size_t)blockIdx.x * kThreads + threadIdx.x;
    const int w = threadIdx.x >> 5;
    count_byte_range(sh_byte[w], codes, n / 2, tid, stride);
    count_byte_range(sh_scale[w], scales, n_blocks, tid, stride);
    __syncthreads();
    // thread t owns byte value t: fold the warps' tables, then the byte counts into the code bins
    unsigned long long cb = 0, cs = 0;
#pragma unroll
    for (int k = 0; k < kWarps; ++k) {
        cb += sh_byte[k][threadIdx.x];
        cs += sh_scale[k][threadIdx.x];
    }
    if (cb) {
        atomicAdd(&sh_code[threadIdx.x & 15], cb);    // element 2j sits in the low nibble
        atomicAdd(&sh_code[threadIdx.x >> 4], cb);
    }
    if (cs) atomicAdd(&scale_hist[threadIdx.x], cs);
    __syncthreads();
    if (threadIdx.x < 16 && sh_code[threadIdx.x]) atomicAdd(&code_hist[threadIdx.x], sh_code[threadIdx.x]);
}

cudaError_t launch_histograms(const uint8_t* codes, const uint8_t* scales, size_t n, int B, unsigned long long* code_hist,
                              unsigned long long* scale_hist, cudaStream_t s) {
    static_assert(kThreads == 256, "one thread per byte value in the fold");
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    size_t want = (n / 32 + kThreads - 1) / kThreads;     // 32 codes per 16-byte load
    if (want == 0) want = 1;
    // a CTA must stay below 2^32 counts per table entry: n / 2 / grid bytes each -- true for any n < 2^40 here
    const size_t cap = (size_t)sm_count(dev) * 4;
    const unsigned grid = (unsigned)(want < cap ? want : cap);
    k_histograms<<<grid, kThreads, 0, s>>>(codes, scales, n, n / (size_t)B, code_hist, scale_hist);
    count_launch();
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// Segment MSE: out[s] = (sum of the block SSEs of segment s) / elems_per_segment.  One CTA per
// segment (grid-stride over segments); thread t adds blocks t, t + 256, ... in order in binary64,
// then a shared-memory halving tree: fixed shape, same bits on every run.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads) k_segment_mse(const float* sse, size_t n_segments, size_t blocks_per_segment,
                                                          double elems_per_segment, double* out) {
    __shared__ double sh[kThreads];
    for (size_t seg = blockIdx.x; seg < n_segments; seg += gridDim.x) {
        const float* p = sse + seg * blocks_per_segment;
        double acc = 0.0;
        for (size_t i = threadIdx.x; i < blocks_per_segment; i += kThreads) acc = __dadd_rn(acc, (double)p[i]);
        sh[threadIdx.x] = acc;
        __syncthreads();
#pragma unroll
        for (int w = kThreads / 2; w > 0; w >>= 1) {
            if (threadIdx.x < w) sh[threadIdx.x] = __dadd_rn(sh[threadIdx.x], sh[threadIdx.x + w]);
            __syncthreads();
        }
        if (threadIdx.x == 0) out[seg] = __ddiv_rn(sh[0], elems_per_segment);
        __syncthreads();
    }
}

cudaError_t launch_segment_mse(const float* sse, size_t n_segments, size_t blocks_per_segment, size_t elems_per_segment,
                               double* out, cudaStream_t s) {
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    const size_t cap = (size_t)sm_count(dev) * 8;
    const unsigned grid = (unsigned)(n_segments < cap ? n_segments : cap);
    k_segment_mse<<<grid, kThreads, 0, s>>>(sse, n_segments, blocks_per_segment, (double)elems_per_segment, out);
    count_launch();
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// Magnitude-interval masking (Appendix, unquantized ablation): entries with lo <= |x| < hi become
// +0, all others pass unchanged.  Elementwise, 16 bytes per thread and trip.
// ------------------------------------------------------------------------------------------------
template <int DT>
__global__ void __launch_bounds__(kThreads) k_mask_interval(const void* x, size_t n, float lo, float hi, void* out) {
    constexpr int VEC = 16 / elem_bytes(DT);
    const size_t n_vec = n / VEC;
    const size_t stride = (size_t)gridDim.x * kThreads;
    for (size_t i = (size_t)blockIdx.x * kThreads + threadIdx.x; i < n_vec; i += stride) {
        uint4 w = __ldcs(static_cast<const uint4*>(x) + i);
        uint32_t* p = reinterpret_cast<uint32_t*>(&w);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            if constexpr (DT == kF32) {
                const float a = fabsf(__uint_as_float(p[k]));
                if (a >= lo && a < hi) p[k] = 0u;
            } else {
                const float a0 = fabsf(__uint_as_float(p[k] << 16)), a1 = fabsf(__uint_as_float(p[k] & 0xFFFF0000u));
                if (a0 >= lo && a0 < hi) p[k] &= 0xFFFF0000u;
                if (a1 >= lo && a1 < hi) p[k] &= 0x0000FFFFu;
            }
        }
        __stcs(static_cast<uint4*>(out) + i, w);
    }
    if (blockIdx.x == 0 && threadIdx.x < (unsigned)(n - n_vec * VEC)) {   // ragged end, scalar
        const size_t e = n_vec * VEC + threadIdx.x;
        if constexpr (DT == kF32) {
            const float v = static_cast<const float*>(x)[e];
            static_cast<float*>(out)[e] = (fabsf(v) >= lo && fabsf(v) < hi) ? 0.0f : v;
        } else {
            const uint16_t h = static_cast<const uint16_t*>(x)[e];
            const float a = fabsf(__uint_as_float((uint32_t)h << 16));
            static_cast<uint16_t*>(out)[e] = (a >= lo && a < hi) ? (uint16_t)0 : h;
        }
    }
}

cudaError_t launch_mask_interval(const void* x, int dtype, size_t n, float lo, float hi, void* out, cudaStream_t s) {
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    size_t want = (n / (16 / elem_bytes(dtype)) + kThreads - 1) / kThreads;
    if (want == 0) want = 1;
    const size_t cap = (size_t)sm_count(dev) * 8;
    const unsigned grid = (unsigned)(want < cap ? want : cap);
    if (dtype == kF32) k_mask_interval<kF32><<<grid, kThreads, 0, s>>>(x, n, lo, hi, out);
    else k_mask_interval<kBF16><<<grid, kThreads, 0, s>>>(x, n, lo, hi, out);
    count_launch();
    return cudaGetLastError();
}

}  // namespace mxq
