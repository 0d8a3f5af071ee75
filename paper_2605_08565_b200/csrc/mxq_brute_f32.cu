// Brute-force scale-search kernels instantiated for f32 input.
#include "mxq_brute.cuh"

namespace mxq {
cudaError_t launch_brute_f32(const QuantArgs& a, int B, int fmt, cudaStream_t s) {
    return launch_brute_dt<kF32, false>(a, B, fmt, s);
}
}  // namespace mxq
