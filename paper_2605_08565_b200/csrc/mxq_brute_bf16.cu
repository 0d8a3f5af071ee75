// Brute-force scale-search kernels instantiated for bf16 input.
#include "mxq_brute.cuh"

namespace mxq {
cudaError_t launch_brute_bf16(const QuantArgs& a, int B, int fmt, cudaStream_t s) {
    return launch_brute_dt<kBF16, false>(a, B, fmt, s);
}
}  // namespace mxq
