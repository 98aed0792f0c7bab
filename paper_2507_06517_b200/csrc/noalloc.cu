// Eviction entry point for callers that must not allocate device memory.
//
// Some hosts of this library cannot call cudaMalloc at the point where the reduction pass runs: a
// serving engine whose memory pool already owns the whole device, a plugin that runs inside another
// framework's allocator lock, or a latency-critical thread where an allocation (an implicit device
// synchronisation) is not acceptable.  For them the scratch memory of the eviction kernels lives in a
// fixed array inside the library image instead of a caller-provided workspace.
#include <mutex>

#include "args.cuh"
#include "common.cuh"

namespace skv {
size_t evict_scratch_needed(const spindlekv_config& cfg, const spindlekv_batch& b, int dtype);
spindlekv_status evict_deep_impl(const spindlekv_config& cfg, const spindlekv_batch& b, const spindlekv_tensor& K,
                                 const spindlekv_tensor& Q, const int32_t* k_ctx, int32_t* keep_idx,
                                 int32_t* keep_cnt, float* scores, void* ws, size_t ws_bytes, cudaStream_t st);
const void* noalloc_scratch_of_current_device();
}  // namespace skv

// The scratch itself: 8 MiB of global memory on every device that loads the library, held until exit.
// In host code this name is only a handle; the device address comes from cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_evict_scratch[SPINDLEKV_NOALLOC_SCRATCH_BYTES];

namespace {
std::mutex g_setup_mu;
void* g_scratch_ptr[skv::kMaxDevices] = {};

// Device address of the scratch array on the current device (looked up once per device).
spindlekv_status scratch_for_current_device(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= skv::kMaxDevices) return SPINDLEKV_CUDA;
  std::lock_guard<std::mutex> lk(g_setup_mu);
  if (!g_scratch_ptr[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_evict_scratch) != cudaSuccess || !ptr) return SPINDLEKV_CUDA;
    g_scratch_ptr[dev] = ptr;
  }
  *out = g_scratch_ptr[dev];
  return SPINDLEKV_OK;
}
}  // namespace

// For spindlekv_poll_status(NULL, ...): the scratch of the current device, or null before the first
// allocation-free call on it.
const void* skv::noalloc_scratch_of_current_device() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= skv::kMaxDevices) return nullptr;
  std::lock_guard<std::mutex> lk(g_setup_mu);
  return g_scratch_ptr[dev];
}

extern "C" spindlekv_status spindlekv_evict_deep_noalloc(const spindlekv_config* cfg, const spindlekv_batch* batch,
                                                         spindlekv_tensor K, spindlekv_tensor Qwin,
                                                         const int32_t* k_ctx, int32_t* keep_idx, int32_t* keep_cnt,
                                                         float* scores, void* stream) {
  // the same checks as spindlekv_evict_deep, all before anything is enqueued
  const spindlekv_status as = skv::evict_args_status(cfg, batch, K, Qwin, k_ctx, keep_idx, keep_cnt, scores);
  if (as != SPINDLEKV_OK) return as;
  // the problem must fit the fixed scratch: say so instead of overrunning it
  if (skv::evict_scratch_needed(*cfg, *batch, K.dtype) > (size_t)SPINDLEKV_NOALLOC_SCRATCH_BYTES)
    return SPINDLEKV_WORKSPACE_TOO_SMALL;
  void* scratch = nullptr;
  spindlekv_status st = scratch_for_current_device(&scratch);
  if (st != SPINDLEKV_OK) return st;
  // the eviction kernels clear the part of the scratch that must start at zero (the status block)
  return skv::evict_deep_impl(*cfg, *batch, K, Qwin, k_ctx, keep_idx, keep_cnt, scores, scratch,
                              (size_t)SPINDLEKV_NOALLOC_SCRATCH_BYTES, (cudaStream_t)stream);
}
