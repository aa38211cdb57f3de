// The fused decode kernel for 3-bit codes.
#include "iq_decode_kernel.cuh"

namespace iq {
cudaError_t launch_decode_b3(const DecodeParams& p, int head_dim, cudaStream_t stream) {
  return p.k_new ? launch_decode_variant<true, 3>(p, head_dim, stream) : launch_decode_variant<false, 3>(p, head_dim, stream);
}
}  // namespace iq
