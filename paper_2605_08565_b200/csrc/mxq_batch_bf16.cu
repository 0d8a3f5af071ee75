// Multi-tensor one-pass quantization kernels instantiated for bf16 input.
#include "mxq_quantize.cuh"

namespace mxq {
cudaError_t launch_quantize_batch_bf16(const QuantArgs& a, int B, int fmt, bool dual, size_t total_rows, cudaStream_t s) {
    return launch_quantize_batch_dt<kBF16>(a, B, fmt, dual, total_rows, s);
}
}  // namespace mxq
