// Fused fake-quantize kernels (quantize + de-quantize in one pass) instantiated for f32 input.
#include "mxq_quantize.cuh"

namespace mxq {
cudaError_t launch_fake_quantize_f32(const QuantArgs& a, int B, int fmt, bool dual, cudaStream_t s) {
    return launch_quantize_dt<kF32, true>(a, B, fmt, dual, s);
}
}  // namespace mxq
