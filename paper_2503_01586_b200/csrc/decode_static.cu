// elitekv_decode_static: decode attention for callers that cannot allocate device memory.
//
// Some hosts of this library may not call cudaMalloc at all: a serving engine that hands its
// whole memory budget to one arena at start-up and forbids later allocations, a plugin running
// inside another framework's step where an allocation would synchronise the device, or code on
// a latency-critical path where the allocator's locks are unwelcome.  elitekv_decode needs a
// caller-provided workspace (work plan + split-K partial results); this variant keeps that
// scratch inside the library image instead, in a fixed-size device array, and allocates
// nothing.  The arithmetic and the kernels are exactly those of elitekv_decode.
#include <mutex>

#include "common.cuh"

namespace {

// The scratch itself.  Every GPU that loads the library holds these bytes until the process
// exits.  In HOST code this name is only a handle for cudaGetSymbolAddress -- it is not a
// device address and must never be passed to a kernel.
static __device__ __align__(256) unsigned char g_static_scratch[ELITEKV_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
void* g_scratch_ptr[kMaxDevices];   // device address of g_static_scratch, per device ordinal
std::mutex g_scratch_mutex;

// Looks the device address up once per device, with that device current.
int scratch_for_current_device(int expected_device, void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return ELITEKV_ERR_CUDA;
  if (dev != expected_device || dev < 0 || dev >= kMaxDevices) return ELITEKV_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (g_scratch_ptr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr)
      return ELITEKV_ERR_CUDA;
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return ELITEKV_OK;
}

}  // namespace

extern "C" int elitekv_decode_static(const elitekv_layer* L, const elitekv_cache* cache,
                                     const void* q_rope, const void* q_abs,
                                     const int32_t* seq_lens, int32_t B, void* out,
                                     elitekv_stream_t stream) {
  if (!L) return ELITEKV_ERR_INVALID_ARG;
  size_t need = 0;
  int rc = elitekv_decode_workspace_size(L, B, &need);
  if (rc != ELITEKV_OK) return rc;
  if (need > (size_t)ELITEKV_STATIC_SCRATCH_BYTES) return ELITEKV_ERR_STATIC_SCRATCH_EXCEEDED;
  void* scratch = nullptr;
  rc = scratch_for_current_device(L->device, &scratch);
  if (rc != ELITEKV_OK) return rc;
  // Nothing in the scratch has to start at zero: the plan kernel rewrites every plan entry and
  // every partial result that is read was written earlier in the same call.
  return elitekv_decode(L, cache, q_rope, q_abs, seq_lens, B, scratch,
                        (size_t)ELITEKV_STATIC_SCRATCH_BYTES, out, stream);
}
