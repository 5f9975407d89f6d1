// diffqkv_decode_static: decode without any caller-provided or freshly allocated scratch memory.
//
// Who needs this: hosts that may not call cudaMalloc at the point where they decode -- an inference
// server whose device memory was handed out in full to a pool at start-up, a plug-in that runs under
// someone else's allocator and has no workspace argument to pass through, a latency-critical loop
// where an allocation would serialise the device.  For them the partial results of the split kernel
// live in a fixed array that is part of the library image itself.
#include <mutex>

#include "common.cuh"

namespace {

constexpr size_t kStaticScratchBytes = 8u << 20;  // 8 MiB, resident on every GPU that loads the library
constexpr int kMaxDevices = 64;

// File-scope device array.  In host code this name is only a handle for the runtime's symbol table,
// never an address a kernel may use; the device address comes from cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

std::mutex g_mutex;
void* g_scratch_ptr[kMaxDevices] = {};

// Device address of the array on the current device; resolved once per device.
cudaError_t scratch_for_current_device(void** out) {
  int dev = -1;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!g_scratch_ptr[dev]) {
    void* ptr = nullptr;
    err = cudaGetSymbolAddress(&ptr, g_static_scratch);
    if (err != cudaSuccess) return err;
    g_scratch_ptr[dev] = ptr;
  }
  *out = g_scratch_ptr[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" diffqkv_status diffqkv_decode_static(const void* q, const diffqkv_cache* cache,
                                                const diffqkv_shape* shape, int32_t num_splits, void* out,
                                                float* lse, int32_t* dev_status, void* stream) {
  if (!shape || !cache) return DIFFQKV_ERR_INVALID_ARG;
  // 0 = nothing to do (batch 0) or arguments diffqkv_decode will refuse: either way it gives the answer below
  const size_t need = diffqkv_decode_workspace_bytes(shape, cache->max_seqlen, num_splits);
  if (need > kStaticScratchBytes) return DIFFQKV_ERR_WORKSPACE;  // beyond the built-in 8 MiB
  void* scratch = nullptr;
  if (scratch_for_current_device(&scratch) != cudaSuccess) return DIFFQKV_ERR_CUDA;
  // Every partial slot the combine kernel reads is written by the split kernel of the same call, so
  // nothing in the array has to start at zero even though it still holds the previous call's data.
  return diffqkv_decode(q, cache, shape, num_splits, scratch, kStaticScratchBytes, out, lse, dev_status, stream);
}
