// Entry points of the fused decode kernel (iq_decode_kernel.cuh): the dispatch over the bit width -- every width is
// compiled in a translation unit of its own -- and the self-test of the bounded wait.
#include "iq_decode_kernel.cuh"

namespace iq {

cudaError_t launch_decode_b2(const DecodeParams& p, int head_dim, cudaStream_t stream);
cudaError_t launch_decode_b3(const DecodeParams& p, int head_dim, cudaStream_t stream);
cudaError_t launch_decode_b4(const DecodeParams& p, int head_dim, cudaStream_t stream);

cudaError_t launch_decode_attention(const DecodeParams& p, int head_dim, cudaStream_t stream) {
  if (p.bits == 2) return launch_decode_b2(p, head_dim, stream);
  if (p.bits == 4) return launch_decode_b4(p, head_dim, stream);
  return launch_decode_b3(p, head_dim, stream);
}

// Self-test of the bounded wait: one warp waits, with `polls` as its limit, on a barrier that nothing completes (no
// copy and no tensor-core work in flight), and reports what the wait returned. polls == 0: the barrier is completed
// before the wait, which then succeeds at its first poll.
__global__ void bounded_wait_selftest_kernel(uint32_t* status, uint32_t polls) {
  __shared__ __align__(8) uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    fence_mbar_init();
    if (polls == 0) mbar_arrive(&bar);
  }
  __syncthreads();
  const bool ok = mbar_wait_bounded(&bar, 0u, polls == 0 ? 16u : polls);
  if (threadIdx.x == 0) {
    if (!ok) atomicOr(&status[0], IQ_STATUS_WAIT_TIMEOUT);
    status[1] = ok ? 0u : polls;
  }
}
cudaError_t launch_bounded_wait_selftest(uint32_t* status, uint32_t polls, cudaStream_t stream) {
  bounded_wait_selftest_kernel<<<1, 32, 0, stream>>>(status, polls);
  return cudaGetLastError();
}

// Groups (independent workers, one partial slot each per piece of an item) the decode kernel runs per CTA.
int decode_groups_per_cta(int head_dim) { return head_dim == 128 ? DecLayout<128>::NG : DecLayout<256>::NG; }
// CTAs the decode kernel keeps resident per SM (it sizes its grid as one CTA per SM).
int decode_ctas_per_sm(int head_dim) { (void)head_dim; return 1; }

}  // namespace iq

