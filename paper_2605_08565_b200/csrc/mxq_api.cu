// C-ABI entry points of libmxq: host-side argument validation and kernel dispatch.
#include <atomic>
#include <cmath>

#include "../../include/mxq.h"
#include "mxq_device.cuh"
#include "mxq_internal.h"

namespace mxq {

static std::atomic<unsigned long long> g_launches{0};
static std::atomic<int> g_brute_prune{0};
static thread_local int tl_cuda_error = 0;

void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

int sm_count(int device) {
    // first-use cache; two threads that race here both store the same value
    static std::atomic<int> cached[kMaxDevices];
    if (device < 0 || device >= kMaxDevices) return 1;
    int n = cached[device].load(std::memory_order_relaxed);
    if (n == 0) {
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || n <= 0) n = 1;
        cached[device].store(n, std::memory_order_relaxed);
    }
    return n;
}

static int cuda_fail(cudaError_t e) {
    tl_cuda_error = (int)e;
    return MXQ_ERR_CUDA;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static bool valid_block(int b) { return b == 2 || b == 4 || b == 8 || b == 16 || b == 32 || b == 64; }

}  // namespace mxq

using namespace mxq;

// Shared by mxq_quantize_ex (codes + scales, optional SSE) and mxq_fake_quantize (x_hat only).
static int quantize_common(const void* x, int dtype, size_t n, int block_size, int scale_fmt, int recipe,
                           float global_scale, const float* d_global_scale, uint8_t* out_codes, uint8_t* out_scales,
                           float* out_block_sse, void* out_xhat, int xhat_dtype, void* cuda_stream,
                           double* d_mse_partials = nullptr, int* n_mse_partials = nullptr) {
    if (!x || (!out_xhat && (!out_codes || !out_scales))) return MXQ_ERR_NULL;
    if (dtype != MXQ_F32 && dtype != MXQ_BF16) return MXQ_ERR_BAD_ENUM;
    if (scale_fmt < MXQ_SF_UE8M0 || scale_fmt > MXQ_SF_UE5M3) return MXQ_ERR_BAD_ENUM;
    if (recipe < MXQ_ABSMAX || recipe > MXQ_ABSMAX_CLIP7) return MXQ_ERR_BAD_ENUM;
    if ((recipe == MXQ_ABSMAX_OCP || recipe == MXQ_ABSMAX_CLIP7) && scale_fmt != MXQ_SF_UE8M0) return MXQ_ERR_BAD_ENUM;
    const bool brute = (recipe == MXQ_BRUTE || recipe == MXQ_BRUTE_PZ);
    if (out_xhat && (brute || (xhat_dtype != MXQ_F32 && xhat_dtype != MXQ_BF16))) return MXQ_ERR_BAD_ENUM;
    if (!valid_block(block_size) || n == 0 || n % (size_t)block_size != 0) return MXQ_ERR_BAD_SHAPE;
    if (!d_global_scale && !(global_scale > 0.0f && std::isfinite(global_scale))) return MXQ_ERR_BAD_SCALE;
    if (!aligned16(x) || !aligned16(out_codes) || !aligned16(out_scales) || !aligned16(out_block_sse) ||
        !aligned16(out_xhat) ||
        (d_global_scale && (reinterpret_cast<uintptr_t>(d_global_scale) & 3u)))
        return MXQ_ERR_ALIGN;

    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    QuantArgs a;
    a.x = x;
    a.first_item = 0;
    a.global_scale = d_global_scale ? 1.0f : global_scale;
    a.d_global_scale = d_global_scale;
    a.codes = out_codes;
    a.scales = out_scales;
    a.block_sse = out_block_sse;
    a.prevent_zero = (recipe == MXQ_ABSMAX_PZ || recipe == MXQ_4O6_PZ || recipe == MXQ_BRUTE_PZ) ? 1 : 0;
    a.pow2_rule = (recipe == MXQ_ABSMAX_OCP) ? kPow2Ocp : (recipe == MXQ_ABSMAX_CLIP7) ? kPow2Clip7 : kPow2Eq1;
    a.xhat = out_xhat;
    a.xhat_dtype = xhat_dtype;
    a.mse_partials = d_mse_partials;
    a.mse_first = 0;
    a.mse_n_partials = n_mse_partials;
    a.batch = nullptr;
    a.n_tensors = 0;

    cudaError_t err;
    if (brute) {
        a.n_items = n / (size_t)block_size;
        // the pruned sweep is a speed option only: same outputs, bit for bit
        if (g_brute_prune.load(std::memory_order_relaxed))
            err = (dtype == MXQ_F32) ? launch_brute_pruned_f32(a, block_size, scale_fmt, s)
                                     : launch_brute_pruned_bf16(a, block_size, scale_fmt, s);
        else
            err = (dtype == MXQ_F32) ? launch_brute_f32(a, block_size, scale_fmt, s)
                                     : launch_brute_bf16(a, block_size, scale_fmt, s);
        return err == cudaSuccess ? MXQ_OK : cuda_fail(err);
    }
    const bool dual = (recipe == MXQ_4O6 || recipe == MXQ_4O6_PZ);
    a.n_items = n / (size_t)block_size;
    if (out_xhat)
        err = (dtype == MXQ_F32) ? launch_fake_quantize_f32(a, block_size, scale_fmt, dual, s)
                                 : launch_fake_quantize_bf16(a, block_size, scale_fmt, dual, s);
    else
        err = (dtype == MXQ_F32) ? launch_quantize_f32(a, block_size, scale_fmt, dual, s)
                                 : launch_quantize_bf16(a, block_size, scale_fmt, dual, s);
    return err == cudaSuccess ? MXQ_OK : cuda_fail(err);
}

extern "C" {

int mxq_quantize_ex(const void* x, int dtype, size_t n, int block_size, int scale_fmt, int recipe, float global_scale,
                    const float* d_global_scale, uint8_t* out_codes, uint8_t* out_scales, float* out_block_sse,
                    void* cuda_stream) {
    if (!out_codes || !out_scales) return MXQ_ERR_NULL;
    return quantize_common(x, dtype, n, block_size, scale_fmt, recipe, global_scale, d_global_scale, out_codes, out_scales,
                           out_block_sse, nullptr, MXQ_F32, cuda_stream);
}

int mxq_fake_quantize(const void* x, int dtype, size_t n, int block_size, int scale_fmt, int recipe, float global_scale,
                      const float* d_global_scale, void* d_out, int out_dtype, void* cuda_stream) {
    if (!d_out) return MXQ_ERR_NULL;
    return quantize_common(x, dtype, n, block_size, scale_fmt, recipe, global_scale, d_global_scale, nullptr, nullptr,
                           nullptr, d_out, out_dtype, cuda_stream);
}

int mxq_quantize_mse(const void* x, int dtype, size_t n, int block_size, int scale_fmt, int recipe, float global_scale,
                     const float* d_global_scale, uint8_t* out_codes, uint8_t* out_scales, float* out_block_sse,
                     double* d_out_mse, void* d_workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!out_codes || !out_scales || !d_out_mse) return MXQ_ERR_NULL;
    if (!d_workspace || workspace_bytes < (size_t)kMsePartials * sizeof(double)) return MXQ_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(d_out_mse) & 7u) || (reinterpret_cast<uintptr_t>(d_workspace) & 7u)) return MXQ_ERR_ALIGN;
    int n_partials = 0;
    const int st = quantize_common(x, dtype, n, block_size, scale_fmt, recipe, global_scale, d_global_scale, out_codes,
                                   out_scales, out_block_sse, nullptr, MXQ_F32, cuda_stream,
                                   static_cast<double*>(d_workspace), &n_partials);
    if (st != MXQ_OK) return st;
    cudaError_t err = launch_mse_final(static_cast<const double*>(d_workspace), n_partials, n, d_out_mse,
                                       static_cast<cudaStream_t>(cuda_stream));
    return err == cudaSuccess ? MXQ_OK : cuda_fail(err);
}

int mxq_quantize_batch(const mxq_tensor_desc* h_descs, const mxq_tensor_desc* d_descs, size_t n_tensors, int dtype,
                       int block_size, int scale_fmt, int recipe, float global_scale, const float* d_global_scale,
                       void* cuda_stream) {
    static_assert(sizeof(mxq_tensor_desc) == sizeof(BatchDesc), "public and internal descriptor layouts agree");
    if (!h_descs || !d_descs) return MXQ_ERR_NULL;
    if (n_tensors == 0 || n_tensors > (size_t)kMaxBatch) return MXQ_ERR_TOO_LARGE;
    if (dtype != MXQ_F32 && dtype != MXQ_BF16) return MXQ_ERR_BAD_ENUM;
    if (scale_fmt < MXQ_SF_UE8M0 || scale_fmt > MXQ_SF_UE5M3) return MXQ_ERR_BAD_ENUM;
    if (recipe < MXQ_ABSMAX || recipe > MXQ_ABSMAX_CLIP7 || recipe == MXQ_BRUTE || recipe == MXQ_BRUTE_PZ) return MXQ_ERR_BAD_ENUM;
    if ((recipe == MXQ_ABSMAX_OCP || recipe == MXQ_ABSMAX_CLIP7) && scale_fmt != MXQ_SF_UE8M0) return MXQ_ERR_BAD_ENUM;
    if (!valid_block(block_size)) return MXQ_ERR_BAD_SHAPE;
    if (!d_global_scale && !(global_scale > 0.0f && std::isfinite(global_scale))) return MXQ_ERR_BAD_SCALE;
    if (!aligned16(d_descs) || (d_global_scale && (reinterpret_cast<uintptr_t>(d_global_scale) & 3u))) return MXQ_ERR_ALIGN;
    const size_t chunk = (size_t)quantize_chunk_elems(dtype, block_size);
    size_t rows = 0;
    for (size_t t = 0; t < n_tensors; ++t) {
        const mxq_tensor_desc& d = h_descs[t];
        if (!d.x || !d.out_codes || !d.out_scales) return MXQ_ERR_NULL;
        if (d.n == 0 || d.n % 64 != 0) return MXQ_ERR_BAD_SHAPE;
        if (!aligned16(d.x) || !aligned16(d.out_codes) || !aligned16(d.out_scales) || !aligned16(d.out_block_sse)) return MXQ_ERR_ALIGN;
        rows += (d.n / chunk + 31) / 32;
    }
    if (rows >= ((size_t)1 << 32)) return MXQ_ERR_TOO_LARGE;
    QuantArgs a;
    a.x = nullptr;
    a.n_items = 0;
    a.first_item = 0;
    a.global_scale = d_global_scale ? 1.0f : global_scale;
    a.d_global_scale = d_global_scale;
    a.codes = nullptr;
    a.scales = nullptr;
    a.block_sse = nullptr;
    a.prevent_zero = (recipe == MXQ_ABSMAX_PZ || recipe == MXQ_4O6_PZ) ? 1 : 0;
    a.pow2_rule = (recipe == MXQ_ABSMAX_OCP) ? kPow2Ocp : (recipe == MXQ_ABSMAX_CLIP7) ? kPow2Clip7 : kPow2Eq1;
    a.xhat = nullptr;
    a.xhat_dtype = MXQ_F32;
    a.mse_partials = nullptr;
    a.mse_first = 0;
    a.mse_n_partials = nullptr;
    a.batch = reinterpret_cast<const BatchDesc*>(d_descs);
    a.n_tensors = (int)n_tensors;
    const bool dual = (recipe == MXQ_4O6 || recipe == MXQ_4O6_PZ);
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t err = (dtype == MXQ_F32) ? launch_quantize_batch_f32(a, block_size, scale_fmt, dual, rows, s)
                                         : launch_quantize_batch_bf16(a, block_size, scale_fmt, dual, rows, s);
    return err == cudaSuccess ? MXQ_OK : cuda_fail(err);
}

int mxq_quantize(const float* x, size_t n, int block_size, int scale_fmt, int recipe, float global_scale,
                 uint8_t* out_codes, uint8_t* out_scales, float* out_block_sse) {
    return mxq_quantize_ex(x, MXQ_F32, n, block_size, scale_fmt, recipe, global_scale, nullptr, out_codes, out_scales,
                           out_block_sse, nullptr);
}

int mxq_tensor_amax(const void* x, int dtype, size_t n, float* d_out_amax, float* d_out_global_scale,
                    void* cuda_stream) {
    if (!x || !d_out_amax) return MXQ_ERR_NULL;
    if (dtype != MXQ_F32 && dtype != MXQ_BF16) return MXQ_ERR_BAD_ENUM;
    if (n == 0) return MXQ_ERR_BAD_SHAPE;
    if (!aligned16(x) || (reinterpret_cast<uintptr_t>(d_out_amax) & 3u) ||
        (reinterpret_cast<uintptr_t>(d_out_global_scale) & 3u))
        return MXQ_ERR_ALIGN;
    cudaError_t err = launch_tensor_amax(x, dtype, n, d_out_amax, d_out_global_scale, static_cast<cudaStream_t>(cuda_stream));
    return err == cudaSuccess ? MXQ_OK : cuda_fail(err);
}

float mxq_global_scale_from_amax(float amax) {
    return (amax > 0.0f && std::isfinite(amax)) ? amax / 2688.0f : 1.0f;
}

size_t mxq_tensor_mse_workspace_bytes(size_t n_blocks) {
    (void)n_blocks;
    return (size_t)kMsePartials * sizeof(double);
}

int mxq_tensor_mse(const float* d_block_sse, size_t n_blocks, size_t n, double* d_out_mse, void* d_workspace,
                   size_t workspace_bytes, void* cuda_stream) {
    if (!d_block_sse || !d_out_mse) return MXQ_ERR_NULL;
    if (n_blocks == 0 || n == 0) return MXQ_ERR_BAD_SHAPE;
    if (!d_workspace || workspace_bytes < mxq_tensor_mse_workspace_bytes(n_blocks)) return MXQ_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(d_block_sse) & 3u) || (reinterpret_cast<uintptr_t>(d_out_mse) & 7u) ||
        (reinterpret_cast<uintptr_t>(d_workspace) & 7u))
        return MXQ_ERR_ALIGN;
    cudaError_t err = launch_tensor_mse(d_block_sse, n_blocks, n, d_out_mse, static_cast<double*>(d_workspace),
                                        static_cast<cudaStream_t>(cuda_stream));
    return err == cudaSuccess ? MXQ_OK : cuda_fail(err);
}

int mxq_tensor_mse_static(const float* d_block_sse, size_t n_blocks, size_t n, double* d_out_mse, void* cuda_stream) {
    if (!d_block_sse || !d_out_mse) return MXQ_ERR_NULL;
    if (n_blocks == 0 || n == 0) return MXQ_ERR_BAD_SHAPE;
    if (n_blocks > MXQ_TENSOR_MSE_STATIC_MAX_BLOCKS) return MXQ_ERR_TOO_LARGE;
    if ((reinterpret_cast<uintptr_t>(d_block_sse) & 3u) || (reinterpret_cast<uintptr_t>(d_out_mse) & 7u))
        return MXQ_ERR_ALIGN;
    cudaError_t err =
        launch_tensor_mse_static(d_block_sse, n_blocks, n, d_out_mse, static_cast<cudaStream_t>(cuda_stream));
    return err == cudaSuccess ? MXQ_OK : cuda_fail(err);
}

int mxq_dequantize_ex(const uint8_t* d_codes, const uint8_t* d_scales, size_t n, int block_size, int scale_fmt,
                      float global_scale, const float* d_global_scale, void* d_out, int out_dtype, void* cuda_stream) {
    if (!d_codes || !d_scales || !d_out) return MXQ_ERR_NULL;
    if (out_dtype != MXQ_F32 && out_dtype != MXQ_BF16) return MXQ_ERR_BAD_ENUM;
    if (scale_fmt < MXQ_SF_UE8M0 || scale_fmt > MXQ_SF_UE5M3) return MXQ_ERR_BAD_ENUM;
    if (!valid_block(block_size) || n == 0 || n % (size_t)block_size != 0) return MXQ_ERR_BAD_SHAPE;
    if (!d_global_scale && !(global_scale > 0.0f && std::isfinite(global_scale))) return MXQ_ERR_BAD_SCALE;
    if (!aligned16(d_codes) || !aligned16(d_out) || (reinterpret_cast<uintptr_t>(d_scales) & 3u) ||
        (reinterpret_cast<uintptr_t>(d_global_scale) & 3u))
        return MXQ_ERR_ALIGN;
    cudaError_t err = launch_dequantize(d_codes, d_scales, n, block_size, scale_fmt, d_global_scale ? 1.0f : global_scale,
                                        d_global_scale, d_out, out_dtype, static_cast<cudaStream_t>(cuda_stream));
    return err == cudaSuccess ? MXQ_OK : cuda_fail(err);
}

int mxq_dequantize(const uint8_t* d_codes, const uint8_t* d_scales, size_t n, int block_size, int scale_fmt,
                   float global_scale, void* d_out, int out_dtype, void* cuda_stream) {
    return mxq_dequantize_ex(d_codes, d_scales, n, block_size, scale_fmt, global_scale, nullptr, d_out, out_dtype,
                             cuda_stream);
}

int mxq_block_clip_sse(const void* x, int dtype, size_t n, int block_size, int scale_fmt, float global_scale,
                       const float* d_global_scale, const uint8_t* d_scales, float* out_clip_sse, void* cuda_stream) {
    if (!x || !d_scales || !out_clip_sse) return MXQ_ERR_NULL;
    if (dtype != MXQ_F32 && dtype != MXQ_BF16) return MXQ_ERR_BAD_ENUM;
    if (scale_fmt < MXQ_SF_UE8M0 || scale_fmt > MXQ_SF_UE5M3) return MXQ_ERR_BAD_ENUM;
    if (!valid_block(block_size) || n == 0 || n % (size_t)block_size != 0) return MXQ_ERR_BAD_SHAPE;
    if (!d_global_scale && !(global_scale > 0.0f && std::isfinite(global_scale))) return MXQ_ERR_BAD_SCALE;
    if (!aligned16(x) || (reinterpret_cast<uintptr_t>(out_clip_sse) & 3u) ||
        (d_global_scale && (reinterpret_cast<uintptr_t>(d_global_scale) & 3u)))
        return MXQ_ERR_ALIGN;
    cudaError_t err = launch_block_clip_sse(x, dtype, n, block_size, scale_fmt, d_global_scale ? 1.0f : global_scale,
                                            d_global_scale, d_scales, out_clip_sse, static_cast<cudaStream_t>(cuda_stream));
    return err == cudaSuccess ? MXQ_OK : cuda_fail(err);
}

int mxq_histograms(const uint8_t* d_codes, const uint8_t* d_scales, size_t n, int block_size,
                   unsigned long long* d_code_hist, unsigned long long* d_scale_hist, void* cuda_stream) {
    if (!d_codes || !d_scales || !d_code_hist || !d_scale_hist) return MXQ_ERR_NULL;
    if (!valid_block(block_size) || n == 0 || n % (size_t)block_size != 0) return MXQ_ERR_BAD_SHAPE;
    if ((reinterpret_cast<uintptr_t>(d_codes) & 3u) || (reinterpret_cast<uintptr_t>(d_code_hist) & 7u) ||
        (reinterpret_cast<uintptr_t>(d_scale_hist) & 7u))
        return MXQ_ERR_ALIGN;
    cudaError_t err = launch_histograms(d_codes, d_scales, n, block_size, d_code_hist, d_scale_hist,
                                        static_cast<cudaStream_t>(cuda_stream));
    return err == cudaSuccess ? MXQ_OK : cuda_fail(err);
}

int mxq_segment_mse(const float* d_block_sse, size_t n_blocks, size_t blocks_per_segment, size_t elems_per_segment,
                    double* d_out_mse, void* cuda_stream) {
    if (!d_block_sse || !d_out_mse) return MXQ_ERR_NULL;
    if (n_blocks == 0 || blocks_per_segment == 0 || elems_per_segment == 0 || n_blocks % blocks_per_segment != 0)
        return MXQ_ERR_BAD_SHAPE;
    if ((reinterpret_cast<uintptr_t>(d_block_sse) & 3u) || (reinterpret_cast<uintptr_t>(d_out_mse) & 7u)) return MXQ_ERR_ALIGN;
    cudaError_t err = launch_segment_mse(d_block_sse, n_blocks / blocks_per_segment, blocks_per_segment, elems_per_segment,
                                         d_out_mse, static_cast<cudaStream_t>(cuda_stream));
    return err == cudaSuccess ? MXQ_OK : cuda_fail(err);
}

int mxq_mask_interval(const void* x, int dtype, size_t n, float lo, float hi, void* d_out, void* cuda_stream) {
    if (!x || !d_out) return MXQ_ERR_NULL;
    if (dtype != MXQ_F32 && dtype != MXQ_BF16) return MXQ_ERR_BAD_ENUM;
    if (n == 0) return MXQ_ERR_BAD_SHAPE;
    if (!(lo >= 0.0f) || !(hi >= lo)) return MXQ_ERR_BAD_SCALE;
    if (!aligned16(x) || !aligned16(d_out)) return MXQ_ERR_ALIGN;
    cudaError_t err = launch_mask_interval(x, dtype, n, lo, hi, d_out, static_cast<cudaStream_t>(cuda_stream));
    return err == cudaSuccess ? MXQ_OK : cuda_fail(err);
}

int mxq_set_option(int option, int value) {
    if (option != MXQ_OPT_BRUTE_PRUNE || (value != 0 && value != 1)) return MXQ_ERR_BAD_ENUM;
    g_brute_prune.store(value, std::memory_order_relaxed);
    return MXQ_OK;
}

int mxq_get_option(int option, int* out_value) {
    if (!out_value) return MXQ_ERR_NULL;
    if (option != MXQ_OPT_BRUTE_PRUNE) return MXQ_ERR_BAD_ENUM;
    *out_value = g_brute_prune.load(std::memory_order_relaxed);
    return MXQ_OK;
}

unsigned long long mxq_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char* mxq_status_string(int status) {
    switch (status) {
    case MXQ_OK: return "ok";
    case MXQ_ERR_NULL: return "a required pointer is NULL";
    case MXQ_ERR_BAD_ENUM: return "dtype, scale format or recipe out of range";
    case MXQ_ERR_BAD_SHAPE: return "n must be a positive multiple of block_size, block_size in {2,4,8,16,32,64}";
    case MXQ_ERR_ALIGN: return "device pointer not sufficiently aligned";
    case MXQ_ERR_BAD_SCALE: return "global_scale must be finite and > 0";
    case MXQ_ERR_WORKSPACE: return "workspace missing or too small";
    case MXQ_ERR_CUDA: return "CUDA call failed (see mxq_last_cuda_error)";
    case MXQ_ERR_TOO_LARGE: return "size exceeds the fixed capacity of this entry point (use the workspace variant)";
    default: return "unknown status";
    }
}

int mxq_last_cuda_error(void) { return tl_cuda_error; }

int mxq_version(void) { return 100; /* 0.1.0 */ }

}  // extern "C"
