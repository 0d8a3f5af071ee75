// Multi-tensor one-pass quantization kernels instantiated for float32 input.
#include "mxq_quantize.cuh"

namespace mxq {
cudaError_t launch_quantize_batch_f32(const QuantArgs& a, int B, int fmt, bool dual, size_t total_rows, cudaStream_t s) {
    return launch_quantize_batch_dt<kF32>(a, B, fmt, dual, total_rows, s);
}
}  // namespace mxq
