// Small kernels around the quantization pass: per-tensor abs-max (first stage of hierarchical
// scaling), deterministic tensor MSE, de-quantization, and a scalar kernel for the few blocks
// that do not fill a whole per-thread chunk.
#include <cuda_bf16.h>

#include <mutex>

#include "mxq_device.cuh"
#include "mxq_internal.h"

namespace mxq {

// ------------------------------------------------------------------------------------------------
// Tensor abs-max: max is exact and order-independent, so the cross-CTA step is an integer
// atomicMax on the bit pattern of the non-negative result (deterministic).
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ float warp_max(float m) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
    return m;
}

// Zeroes the running maximum and, when a tensor scale is wanted, the word that first counts the CTAs
// that have finished and then receives the scale.
__global__ void k_amax_init(uint32_t* amax_bits, uint32_t* g_word) {
    wait_for_prior_grid();
    release_dependents();
    *amax_bits = 0u;
    if (g_word) *g_word = 0u;
}

// One CTA reads tiles of U x 256 sixteen-byte vectors (U independent loads per thread in flight).  The
// last CTA to finish (a count in g_word) turns the maximum into g = amax / (6 * 448), the tensor
// maximum mapped to the top of FP4 times the top of E4M3, and stores it over the count.  Loads are
// streaming (evict-first): reading with the default policy, so that the quantize pass that follows finds
// the tensor in L2, was measured on 33 to 117 MB tensors and gains nothing (that pass is not DRAM-bound
// enough at those sizes), while it slows this kernel by 5 %.
template <int DT>
__global__ void __launch_bounds__(kThreads) k_tensor_amax(const void* x, size_t n, uint32_t* out_bits, uint32_t* g_word) {
    constexpr int VEC = 16 / elem_bytes(DT);
    constexpr int U = 4;
    const size_t n_vec = n / VEC;
    const size_t tile = (size_t)U * kThreads;
    const uint4* p = static_cast<const uint4*>(x);
    {   // while the kernel before this one drains: ask L2 for this thread's first vector (no architectural effect)
        const size_t first = (size_t)blockIdx.x * tile + threadIdx.x;
        if (first < n_vec) asm volatile("prefetch.global.L2 [%0];" ::"l"(p + first));
    }
    wait_for_prior_grid();
    release_dependents();
    float m = 0.0f;
    uint32_t a16 = 0;   // bf16: magnitudes order like their 15-bit patterns, packed unsigned 16-bit max
    for (size_t base = (size_t)blockIdx.x * tile; base < n_vec; base += (size_t)gridDim.x * tile) {
        uint4 w[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const size_t i = base + (size_t)u * kThreads + threadIdx.x;
            w[u] = make_uint4(0u, 0u, 0u, 0u);
            if (i < n_vec) w[u] = __ldcs(p + i);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if constexpr (DT == kF32) {
                m = fmaxf(fmaxf(m, fabsf(__uint_as_float(w[u].x))), fabsf(__uint_as_float(w[u].y)));
                m = fmaxf(fmaxf(m, fabsf(__uint_as_float(w[u].z))), fabsf(__uint_as_float(w[u].w)));
            } else {
                a16 = __vmaxu2(a16, __vmaxu2(w[u].x & 0x7FFF7FFFu, w[u].y & 0x7FFF7FFFu));
                a16 = __vmaxu2(a16, __vmaxu2(w[u].z & 0x7FFF7FFFu, w[u].w & 0x7FFF7FFFu));
            }
        }
    }
    if constexpr (DT == kBF16) m = fmaxf(__uint_as_float(a16 << 16), __uint_as_float(a16 & 0xFFFF0000u));
    if (blockIdx.x == 0 && threadIdx.x < (unsigned)(n - n_vec * VEC)) {  // ragged end, scalar
        const size_t i = n_vec * VEC + threadIdx.x;
        float v;
        if constexpr (DT == kF32) v = static_cast<const float*>(x)[i];
        else v = __uint_as_float((uint32_t) static_cast<const uint16_t*>(x)[i] << 16);
        m = fmaxf(m, fabsf(v));
    }
    __shared__ float warp_m[kThreads / 32];
    m = warp_max(m);
    if ((threadIdx.x & 31) == 0) warp_m[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x < 32) {
        m = threadIdx.x < kThreads / 32 ? warp_m[threadIdx.x] : 0.0f;
        m = warp_max(m);
        if (threadIdx.x == 0) {
            atomicMax(out_bits, __float_as_uint(m));
            if (g_word) {
                __threadfence();
                if (atomicAdd(g_word, 1u) == gridDim.x - 1) {   // every CTA's maximum is in: this one writes the scale
                    __threadfence();
                    const float a = __uint_as_float(atomicMax(out_bits, 0u));
                    *reinterpret_cast<float*>(g_word) = (a > 0.0f && a <= 3.402823466e38f) ? __fdiv_rn(a, 2688.0f) : 1.0f;
                }
            }
        }
    }
}

cudaError_t launch_tensor_amax(const void* x, int dtype, size_t n, float* d_amax, float* d_g, cudaStream_t s) {
    uint32_t* amax_bits = reinterpret_cast<uint32_t*>(d_amax);
    uint32_t* g_word = reinterpret_cast<uint32_t*>(d_g);
    cudaError_t err = launch_pdl(k_amax_init, 1u, 1u, 0, s, amax_bits, g_word);
    count_launch();
    if (err != cudaSuccess) return err;
    int dev = 0;
    err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    const size_t n_vec = n / (16 / elem_bytes(dtype));
    size_t want = (n_vec + 4 * kThreads - 1) / (4 * kThreads);
    if (want == 0) want = 1;
    const size_t cap = (size_t)sm_count(dev) * 8;
    const unsigned grid = (unsigned)(want < cap ? want : cap);
    if (dtype == kF32) err = launch_pdl(k_tensor_amax<kF32>, grid, (unsigned)kThreads, 0, s, x, n, amax_bits, g_word);
    else err = launch_pdl(k_tensor_amax<kBF16>, grid, (unsigned)kThreads, 0, s, x, n, amax_bits, g_word);
    count_launch();
    return err;
}

// ------------------------------------------------------------------------------------------------
// Tensor MSE: two-level tree of fixed shape in binary64.  Level 1: P = min(1024, ceil(nb/256))
// CTAs, CTA p sums the contiguous slice [p*L, (p+1)*L), L = ceil(nb/P): thread t adds elements
// t, t+256, ... in order, then a shared-memory halving tree.  Level 2: one CTA, halving tree over
// the P partials, divided by n.
// ------------------------------------------------------------------------------------------------
template <int T>
__device__ __forceinline__ double cta_tree_sum(double v, double* sh) {
    sh[threadIdx.x] = v;
    __syncthreads();
#pragma unroll
    for (int w = T / 2; w > 0; w >>= 1) {
        if (threadIdx.x < w) sh[threadIdx.x] = __dadd_rn(sh[threadIdx.x], sh[threadIdx.x + w]);
        __syncthreads();
    }
    return sh[0];
}

__global__ void __launch_bounds__(kThreads) k_mse_partial(const float* sse, size_t nb, size_t slice, double* partials) {
    __shared__ double sh[kThreads];
    wait_for_prior_grid();
    release_dependents();
    const size_t lo = (size_t)blockIdx.x * slice;
    const size_t hi = (lo + slice < nb) ? lo + slice : nb;
    double acc = 0.0;
    for (size_t i = lo + threadIdx.x; i < hi; i += kThreads) acc = __dadd_rn(acc, (double)__ldcs(sse + i));
    const double total = cta_tree_sum<kThreads>(acc, sh);
    if (threadIdx.x == 0) partials[blockIdx.x] = total;
}

__global__ void __launch_bounds__(kMsePartials) k_mse_final(const double* partials, int n_partials, double n, double* out) {
    __shared__ double sh[kMsePartials];
    wait_for_prior_grid();
    release_dependents();
    const double v = (int)threadIdx.x < n_partials ? partials[threadIdx.x] : 0.0;
    const double total = cta_tree_sum<kMsePartials>(v, sh);
    if (threadIdx.x == 0) *out = __ddiv_rn(total, n);
}

cudaError_t launch_tensor_mse(const float* d_sse, size_t n_blocks, size_t n, double* d_out, double* d_partials,
                              cudaStream_t s) {
    size_t P = (n_blocks + kThreads - 1) / kThreads;
    if (P > (size_t)kMsePartials) P = kMsePartials;
    const size_t slice = (n_blocks + P - 1) / P;
    // staged launches: the launch latency of these two small kernels comes off the critical path
    cudaError_t err = launch_pdl(k_mse_partial, (unsigned)P, kThreads, 0, s, d_sse, n_blocks, slice, d_partials);
    count_launch();
    if (err != cudaSuccess) return err;
    err = launch_pdl(k_mse_final, 1u, (unsigned)kMsePartials, 0, s, (const double*)d_partials, (int)P, (double)n, d_out);
    count_launch();
    return err;
}

cudaError_t launch_mse_final(const double* d_partials, int n_partials, size_t n, double* d_out, cudaStream_t s) {
    cudaError_t err = launch_pdl(k_mse_final, 1u, (unsigned)kMsePartials, 0, s, d_partials, n_partials, (double)n, d_out);
    count_launch();
    return err;
}

// ------------------------------------------------------------------------------------------------
// De-quantization: x_hat = fl32(grid(code) * D), D = fl32(S * g).  One thread per 8 elements.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ float decode_scale(int fmt, int c, float g) {
    if (c >= num_codes(fmt)) return __uint_as_float(0x7FC00000u);
    return __fmul_rn(scale_value(fmt, c), g);
}

// A unit is the run of elements whose results one thread writes with ONE 16-byte store, so that a
// warp's store covers 512 contiguous bytes: 8 elements for bf16 output, 4 for fp32 output.  Four
// units per thread and trip, and the loads of the next trip issued before this trip's stores, keep
// eight independent loads in flight.  Measured on 134 M elements: 110 to 115 us for fp32 output (5.4 TB/s of
// codes + scales + output; a plain fill of the same output alone takes 82 us) whatever was tried -- plain
// instead of streaming stores, 4, 8 or 16 resident CTAs per SM, grid-stride or CTA-contiguous tiles, with
// or without the table and the early loads; those two shorten B = 2 by about 5 % and were kept.
template <int ODT>
__global__ void __launch_bounds__(kThreads) k_dequantize(const uint8_t* codes, const uint8_t* scales, size_t n,
                                                         int log2B, int fmt, float g_host, const float* d_g, void* out) {
    wait_for_prior_grid();
    release_dependents();
    const float g = d_g ? *d_g : g_host;   // device-resident tensor scale (written by an earlier kernel of the stream)
    // decode scales of all 256 codes, one per thread: a table read replaces a dozen instructions per unit
    __shared__ float Dtab[256];
    Dtab[threadIdx.x] = decode_scale(fmt, (int)threadIdx.x, g);
    __syncthreads();
    constexpr int E = (ODT == kF32) ? 4 : 8;      // elements per unit
    constexpr int LOG2E = (ODT == kF32) ? 2 : 3;
    constexpr int U = 4;
    const size_t n_units = n / E;
    const size_t stride = (size_t)gridDim.x * kThreads;
    // the loads of the next trip are issued before the arithmetic and the stores of this one
    auto load_trip = [&](size_t first, uint32_t (&w)[U], uint32_t (&sc)[U]) {
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const size_t i = first + (size_t)u * kThreads;
            w[u] = 0;
            sc[u] = 0;
            if (i < n_units) {
                if constexpr (E == 8) w[u] = __ldcs(reinterpret_cast<const uint32_t*>(codes) + i);
                else w[u] = __ldcs(reinterpret_cast<const uint16_t*>(codes) + i);
                // the scale codes of the unit's blocks (one byte when a block holds the whole unit)
                if (log2B >= LOG2E) sc[u] = scales[(i << LOG2E) >> log2B];
                else if (E >> log2B == 2) sc[u] = reinterpret_cast<const uint16_t*>(scales)[i];
                else sc[u] = reinterpret_cast<const uint32_t*>(scales)[i];
            }
        }
    };
    // a CTA works on tiles of U x 256 consecutive units (16 KB of fp32 output), tiles b, b + grid, ...
    size_t base = (size_t)blockIdx.x * (U * kThreads) + threadIdx.x;
    uint32_t w[U], sc[U];
    load_trip(base, w, sc);
    for (; base < n_units; base += stride * U) {
        uint32_t wn[U], scn[U];
        load_trip(base + stride * U, wn, scn);
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const size_t i = base + (size_t)u * kThreads;
            if (i >= n_units) continue;
            float q[8];
            unpack_e2m1x8(w[u], q);
            float xh[E];
            if (log2B >= LOG2E) {
                const float D = Dtab[sc[u]];
#pragma unroll
                for (int k = 0; k < E; ++k) xh[k] = __fmul_rn(q[k], D);
            } else {
#pragma unroll
                for (int k = 0; k < E; ++k)
                    xh[k] = __fmul_rn(q[k], Dtab[(sc[u] >> (8 * (k >> log2B))) & 0xFFu]);
            }
            if constexpr (ODT == kF32) {
                __stcs(static_cast<float4*>(out) + i, make_float4(xh[0], xh[1], xh[2], xh[3]));
            } else {
                uint32_t h[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const __nv_bfloat162 b = __floats2bfloat162_rn(xh[2 * k], xh[2 * k + 1]);
                    h[k] = *reinterpret_cast<const uint32_t*>(&b);
                }
                __stcs(static_cast<uint4*>(out) + i, make_uint4(h[0], h[1], h[2], h[3]));
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            w[u] = wn[u];
            sc[u] = scn[u];
        }
    }
    // ragged end (n not a multiple of the unit; only possible for block sizes 2 and 4)
    if (blockIdx.x == 0 && threadIdx.x < (unsigned)(n - n_units * E)) {
        const size_t e = n_units * E + threadIdx.x;
        const uint32_t c4 = (codes[e >> 1] >> ((e & 1) ? 4 : 0)) & 15u;
        float q[8];
        unpack_e2m1x8(c4, q);
        const float xh = __fmul_rn(q[0], Dtab[scales[e >> log2B]]);
        if constexpr (ODT == kF32) static_cast<float*>(out)[e] = xh;
        else static_cast<__nv_bfloat16*>(out)[e] = __float2bfloat16_rn(xh);
    }
}

cudaError_t launch_dequantize(const uint8_t* codes, const uint8_t* scales, size_t n, int B, int fmt, float g,
                              const float* d_g, void* out, int out_dtype, cudaStream_t s) {
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    int log2B = 0;
    while ((1 << log2B) < B) ++log2B;
    size_t want = ((n >> (out_dtype == kF32 ? 2 : 3)) / 4 + kThreads - 1) / kThreads;   // four units per thread
    if (want == 0) want = 1;
    const size_t cap = (size_t)sm_count(dev) * 8;
    const unsigned grid = (unsigned)(want < cap ? want : cap);
    if (out_dtype == kF32) err = launch_pdl(k_dequantize<kF32>, grid, kThreads, 0, s, codes, scales, n, log2B, fmt, g, d_g, out);
    else err = launch_pdl(k_dequantize<kBF16>, grid, kThreads, 0, s, codes, scales, n, log2B, fmt, g, d_g, out);
    count_launch();
    return err;
}

// ------------------------------------------------------------------------------------------------
// Scalar abs-max / 4-over-6 for the blocks past the last whole per-thread chunk (block sizes up to
// 16, fewer than 16 blocks).
// Same arithmetic as the one-pass kernels, general quotient only.
// ------------------------------------------------------------------------------------------------
template <int FMT>
__device__ float tail_eval(const float* v, int B, int c, float g, uint8_t* codes_out) {
    const float D = __fmul_rn(scale_value(FMT, c), g);
    float s = 0.0f;
    for (int i = 0; i < B; i += 2) {
        const float t0 = quotient_general(v[i], D), t1 = quotient_general(v[i + 1], D);
        if (codes_out) codes_out[i >> 1] = (uint8_t)pack_e2m1x2(t0, t1);
        const float2 q = round_e2m1x2(t0, t1);
        const float e0 = __fmaf_rn(-q.x, D, v[i]);
        s = __fmaf_rn(e0, e0, s);
        const float e1 = __fmaf_rn(-q.y, D, v[i + 1]);
        s = __fmaf_rn(e1, e1, s);
    }
    return s;
}

template <int FMT>
__global__ void k_quantize_tail(QuantArgs p, int dtype, int B, int dual) {
    const size_t b = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    float my_sse = 0.0f;
    if (b < p.n_items) {
    const size_t blk = p.first_item + b;
    const float g = p.d_global_scale ? *p.d_global_scale : p.global_scale;
    float v[16];
    float amax = 0.0f;
    for (int i = 0; i < B; ++i) {
        const size_t e = blk * B + i;
        v[i] = dtype == kF32 ? static_cast<const float*>(p.x)[e]
                             : __uint_as_float((uint32_t) static_cast<const uint16_t*>(p.x)[e] << 16);
        amax = fmaxf(amax, fabsf(v[i]));
    }
    const bool pz = p.prevent_zero && FMT != kUE8M0;
    const float u = __fdiv_rn(amax, g);
    int c = (FMT == kUE8M0 && p.pow2_rule != kPow2Eq1) ? pow2_rule_code(u, p.pow2_rule) : round_scale<FMT>(__fdiv_rn(u, 6.0f));
    if (pz) c = max(c, 1);
    float s = tail_eval<FMT>(v, B, c, g, nullptr);
    if (dual) {
        int c4 = round_scale<FMT>(__fdiv_rn(u, 4.0f));
        if (pz) c4 = max(c4, 1);
        const float s4 = tail_eval<FMT>(v, B, c4, g, nullptr);
        if (s4 < s) { s = s4; c = c4; }
    }
    uint8_t packed[8];
    tail_eval<FMT>(v, B, c, g, packed);
    if (p.codes)
        for (int i = 0; i < B / 2; ++i) p.codes[blk * (B / 2) + i] = packed[i];
    if (p.scales) p.scales[blk] = (uint8_t)c;
    if (p.block_sse) p.block_sse[blk] = s;
    if (p.xhat) {
        const float D = __fmul_rn(scale_value(FMT, c), g);
        for (int i = 0; i < B; ++i) {
            float q[8];
            unpack_e2m1x8((uint32_t)((packed[i >> 1] >> ((i & 1) ? 4 : 0)) & 15u), q);
            const float xh = __fmul_rn(q[0], D);
            if (p.xhat_dtype == kF32) static_cast<float*>(p.xhat)[blk * B + i] = xh;
            else static_cast<__nv_bfloat16*>(p.xhat)[blk * B + i] = __float2bfloat16_rn(xh);
        }
    }
    my_sse = s;
    }
    // fused tensor-MSE partial sum: the kernel is one warp, every lane takes part (idle lanes add 0)
    if (p.mse_partials != nullptr) warp_sum_to_partial(p, my_sse);
}

cudaError_t launch_quantize_tail(const QuantArgs& a, int dtype, int B, int fmt, bool dual, cudaStream_t s) {
    if (B > 16) return cudaErrorInvalidValue;
    const unsigned grid = (unsigned)((a.n_items + 31) / 32);
    switch (fmt) {
    case kUE8M0: k_quantize_tail<kUE8M0><<<grid, 32, 0, s>>>(a, dtype, B, dual ? 1 : 0); break;
    case kUE4M3: k_quantize_tail<kUE4M3><<<grid, 32, 0, s>>>(a, dtype, B, dual ? 1 : 0); break;
    default: k_quantize_tail<kUE5M3><<<grid, 32, 0, s>>>(a, dtype, B, dual ? 1 : 0); break;
    }
    count_launch();
    return cudaGetLastError();
}

}  // namespace mxq

// ------------------------------------------------------------------------------------------------
// Tensor MSE for callers that cannot provide scratch memory: the first-level partial sums live in
// a file-scope device array instead of a caller workspace.  Every GPU that loads the library
// carries these 8 KiB until the process exits.  In host code the array's name is only a handle
// for the runtime, so its device address is looked up once per device (with that device current)
// and handed to the same two kernels as the workspace variant.  Nothing in the array has to start
// at zero: the first kernel writes every partial the second one reads.
// ------------------------------------------------------------------------------------------------
namespace mxq {

static __device__ __align__(256) double g_mse_static_partials[kMsePartials];

cudaError_t launch_tensor_mse_static(const float* d_sse, size_t n_blocks, size_t n, double* d_out, cudaStream_t s) {
    static std::mutex mu;
    static double* scratch_of_device[kMaxDevices] = {nullptr};
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    double* scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(mu);
        scratch = scratch_of_device[dev];
        if (scratch == nullptr) {  // first call on this device: resolve the symbol to a device address
            void* p = nullptr;
            err = cudaGetSymbolAddress(&p, g_mse_static_partials);
            if (err != cudaSuccess) return err;
            if (p == nullptr) return cudaErrorInvalidSymbol;
            scratch = static_cast<double*>(p);
            scratch_of_device[dev] = scratch;
        }
    }
    return launch_tensor_mse(d_sse, n_blocks, n, d_out, scratch, s);
}

}  // namespace mxq
