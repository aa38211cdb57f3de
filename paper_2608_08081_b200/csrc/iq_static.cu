// Decode entry point for callers that cannot allocate device memory.
//
// iq_decode_attention needs scratch for the per-split partial results, and normally the caller allocates
// it. Some callers cannot: code running inside a CUDA-graph capture or under a framework allocator that
// must not be re-entered, a plugin that is handed only its input and output buffers, or an embedding whose
// memory budget is fixed at load time. For them this file keeps the scratch in a fixed-size array that
// is part of the library image: every GPU that loads the library holds IQ_STATIC_SCRATCH_BYTES of device
// memory for it until the process exits.
//
// In host code the name of a __device__ array is only a host-side stand-in, not a device address, so the
// address is looked up once per device with cudaGetSymbolAddress (with that device current) and the
// pointer is what the kernels receive. The looked-up address is kept for the life of the process: it does
// not survive a cudaDeviceReset of that device, after which this entry point must not be used again.
#include <mutex>

#include "iq_common.cuh"
#include "iq_kernels.h"

namespace {

constexpr size_t kScratchFloats = IQ_STATIC_SCRATCH_BYTES / sizeof(float);
static __device__ __align__(256) float g_iq_static_scratch[kScratchFloats];

constexpr int kMaxDevices = 64;
float* g_scratch_ptr[kMaxDevices] = {};
std::mutex g_scratch_mutex;

// Device address of the scratch array on the current device; resolved on the first call per device.
int scratch_for_current_device(float** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return IQ_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_ptr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_iq_static_scratch) != cudaSuccess || !p) return IQ_ERR_CUDA;
    g_scratch_ptr[dev] = static_cast<float*>(p);
  }
  *out = g_scratch_ptr[dev];
  return IQ_OK;
}

}  // namespace

extern "C" {

size_t iq_static_scratch_bytes(void) { return IQ_STATIC_SCRATCH_BYTES; }

int iq_decode_attention_static(const iq_shape* shape, const float* rot_dev, const iq_codebook* codebook, const void* q,
                               const iq_cache* cache, const int32_t* seq_lens_dev, int32_t num_splits, void* out,
                               int32_t out_is_fp16, float* lse_out, uint32_t* status_dev, void* stream) {
  if (!shape) return IQ_ERR_NULL;
  // what the merge would refuse after the decode kernel has been enqueued is refused here instead
  if (!out) return IQ_ERR_NULL;
  if ((reinterpret_cast<uintptr_t>(out) & 15u) != 0) return IQ_ERR_ALIGN;
  if (num_splits < 1) return IQ_ERR_SHAPE;
  if (shape->batch < 0 || shape->n_q_heads <= 0 || (shape->head_dim != 128 && shape->head_dim != 256)) return IQ_ERR_SHAPE;
  // partials: acc [B][H_q][S][d] followed by (m, l) [B][H_q][S][2]
  const size_t heads = (size_t)shape->batch * (size_t)shape->n_q_heads * (size_t)num_splits;
  const size_t need = heads * ((size_t)shape->head_dim + 2);
  if (need > kScratchFloats) return IQ_ERR_LIMIT;
  float* scratch = nullptr;
  int rc = scratch_for_current_device(&scratch);
  if (rc != IQ_OK) return rc;
  float* part_acc = scratch;
  float* part_ml = scratch + heads * (size_t)shape->head_dim;
  // Every split of every head is rewritten by the decode kernel on each call (empty splits included), so
  // nothing in the shared array has to be cleared between calls.
  rc = iq_decode_attention(shape, rot_dev, codebook, q, cache, seq_lens_dev, num_splits, part_acc, part_ml, nullptr,
                           status_dev, stream);
  if (rc != IQ_OK) return rc;
  return iq_combine_splits(shape, rot_dev, num_splits, part_acc, part_ml, nullptr, out, out_is_fp16, lse_out, nullptr, stream);
}

}  // extern "C"
