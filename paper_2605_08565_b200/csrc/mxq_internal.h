// Host-side declarations shared by the translation units of libmxq (not part of the public ABI).
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace mxq {

constexpr int kMaxDevices = 64;

// Arguments of the quantization kernels.  The launchers receive n_items = number of blocks and
// hand their kernels n_items = what one thread owns per loop trip (chunks of blocks, or blocks).
// Power-of-two scale rules (UE8M0): Eq. 1 as printed; the OCP wording; the [3.5, 7) target.
enum { kPow2Eq1 = 0, kPow2Ocp = 1, kPow2Clip7 = 2 };

// One tensor of a multi-tensor launch (device-resident array; the public mxq_tensor_desc has this layout).
struct BatchDesc {
    const void* x;
    uint8_t* codes;
    uint8_t* scales;
    float* block_sse;   // may be NULL
    size_t n;           // elements
};
constexpr int kMaxBatch = 1024;   // tensors per multi-tensor launch

struct QuantArgs {
    const void* x;
    size_t n_items;
    size_t first_item;            // tail kernel only: index of the first block it handles
    float global_scale;
    const float* d_global_scale;  // overrides global_scale when non-NULL
    uint8_t* codes;
    uint8_t* scales;
    float* block_sse;             // may be NULL
    int prevent_zero;
    int pow2_rule;                // UE8M0 only: which power-of-two rule (kPow2Eq1, kPow2Ocp, kPow2Clip7)
    void* xhat;                   // fused fake-quantize output (codes / scales may then be NULL), or NULL
    int xhat_dtype;
    // fused tensor-MSE partial sums (mxq_quantize_mse), or NULL: CTA i of the main kernel stores the
    // binary64 sum of the block SSEs it produced in mse_partials[mse_first + i]; the tail kernel (one
    // warp) stores its sum in mse_partials[mse_first]
    double* mse_partials;
    int mse_first;
    int* mse_n_partials;          // host: receives how many partials the launches of this call write (or NULL)
    // multi-tensor launch (mxq_quantize_batch): device array of n_tensors descriptors; x, codes, scales,
    // block_sse and n_items above are then unused
    const BatchDesc* batch;
    int n_tensors;
};

int sm_count(int device);

// Launch with programmatic stream serialization: the grid may be staged while the kernel before
// it in the stream still runs.  EVERY kernel launched this way calls wait_for_prior_grid() before
// its first access to global memory; the wait returns once that kernel has completed and its
// writes are visible (at once when there is nothing to wait for).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), unsigned grid, unsigned block, size_t smem, cudaStream_t stream,
                              Args... args) {
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
void count_launch();

cudaError_t launch_quantize_f32(const QuantArgs& a, int B, int fmt, bool dual, cudaStream_t s);
cudaError_t launch_quantize_bf16(const QuantArgs& a, int B, int fmt, bool dual, cudaStream_t s);
// Multi-tensor launch: a.batch / a.n_tensors set; total_rows = sum over tensors of ceil(chunks / 32),
// chunks = n / quantize_chunk_elems(dtype, B).
cudaError_t launch_quantize_batch_f32(const QuantArgs& a, int B, int fmt, bool dual, size_t total_rows, cudaStream_t s);
cudaError_t launch_quantize_batch_bf16(const QuantArgs& a, int B, int fmt, bool dual, size_t total_rows, cudaStream_t s);
// Elements one thread of the one-pass kernels handles per trip (at least 64 bytes and one block).
__host__ __device__ constexpr int quantize_chunk_elems(int dtype, int B) { return dtype == 0 ? (B > 16 ? B : 16) : (B > 32 ? B : 32); }
cudaError_t launch_fake_quantize_f32(const QuantArgs& a, int B, int fmt, bool dual, cudaStream_t s);
cudaError_t launch_fake_quantize_bf16(const QuantArgs& a, int B, int fmt, bool dual, cudaStream_t s);
cudaError_t launch_brute_f32(const QuantArgs& a, int B, int fmt, cudaStream_t s);
cudaError_t launch_brute_bf16(const QuantArgs& a, int B, int fmt, cudaStream_t s);
cudaError_t launch_brute_pruned_f32(const QuantArgs& a, int B, int fmt, cudaStream_t s);
cudaError_t launch_brute_pruned_bf16(const QuantArgs& a, int B, int fmt, cudaStream_t s);
// Scalar kernel for the few blocks that do not fill a whole chunk (abs-max and 4-over-6 only).
cudaError_t launch_quantize_tail(const QuantArgs& a, int dtype, int B, int fmt, bool dual, cudaStream_t s);

cudaError_t launch_tensor_amax(const void* x, int dtype, size_t n, float* d_amax, float* d_g, cudaStream_t s);
cudaError_t launch_tensor_mse(const float* d_sse, size_t n_blocks, size_t n, double* d_out, double* d_partials,
                              cudaStream_t s);
// Same reduction with the first-level partials in a library-owned device array (no workspace).
cudaError_t launch_tensor_mse_static(const float* d_sse, size_t n_blocks, size_t n, double* d_out, cudaStream_t s);
cudaError_t launch_dequantize(const uint8_t* codes, const uint8_t* scales, size_t n, int B, int fmt, float g,
                              const float* d_g, void* out, int out_dtype, cudaStream_t s);

cudaError_t launch_block_clip_sse(const void* x, int dtype, size_t n, int B, int fmt, float g, const float* d_g,
                                  const uint8_t* scales, float* out, cudaStream_t s);
cudaError_t launch_histograms(const uint8_t* codes, const uint8_t* scales, size_t n, int B, unsigned long long* code_hist,
                              unsigned long long* scale_hist, cudaStream_t s);
cudaError_t launch_segment_mse(const float* sse, size_t n_segments, size_t blocks_per_segment, size_t elems_per_segment,
                               double* out, cudaStream_t s);

cudaError_t launch_mask_interval(const void* x, int dtype, size_t n, float lo, float hi, void* out, cudaStream_t s);

constexpr int kMsePartials = 1024;  // fixed first-level width of the MSE tree
// Second level of the tensor-MSE tree alone: out = (sum of n_partials <= kMsePartials partials) / n.
cudaError_t launch_mse_final(const double* d_partials, int n_partials, size_t n, double* d_out, cudaStream_t s);

}  // namespace mxq
