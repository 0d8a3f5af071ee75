// One-pass quantization kernels instantiated for f32 input.
#include "mxq_quantize.cuh"

namespace mxq {
cudaError_t launch_quantize_f32(const QuantArgs& a, int B, int fmt, bool dual, cudaStream_t s) {
    return launch_quantize_dt<kF32, false>(a, B, fmt, dual, s);
}
}  // namespace mxq
