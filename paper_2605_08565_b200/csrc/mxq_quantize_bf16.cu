// One-pass quantization kernels instantiated for bf16 input.
#include "mxq_quantize.cuh"

namespace mxq {
cudaError_t launch_quantize_bf16(const QuantArgs& a, int B, int fmt, bool dual, cudaStream_t s) {
    return launch_quantize_dt<kBF16, false>(a, B, fmt, dual, s);
}
}  // namespace mxq
