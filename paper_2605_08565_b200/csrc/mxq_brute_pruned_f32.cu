// Brute-force scale-search kernels with the pruned sweep, instantiated for binary32 input.
#include "mxq_brute.cuh"

namespace mxq {
cudaError_t launch_brute_pruned_f32(const QuantArgs& a, int B, int fmt, cudaStream_t s) {
    return launch_brute_dt<kF32, true>(a, B, fmt, s);
}
}  // namespace mxq
