// The fused decode kernel for 2-bit codes.
#include "iq_decode_kernel.cuh"

namespace iq {
cudaError_t launch_decode_b2(const DecodeParams& p, int head_dim, cudaStream_t stream) {
  if (p.k_new) return cudaErrorNotSupported;  // (refused by the C ABI before it gets here)
  return launch_decode_variant<false, 2>(p, head_dim, stream);
}
}  // namespace iq
