// thanos_prune_layer_noalloc: the block sweep for callers that cannot hand over a workspace.
//
// The sweep's scratch (per-block matrices, the bf16 planes of the update operands, histogram,
// sweep state, tie prefixes, row lists, the keys copied out of the selection window, and the fp32
// working copy for 16-bit weights) lives in one fixed array in the library's device image instead
// of a caller buffer.  Everything else is the ordinary sweep.
#include <mutex>

#include "common.cuh"

namespace thanos {
size_t prune_workspace_bytes(int64_t c, int64_t b, int32_t B, thanos_dtype_t dtype);
thanos_status_t check_prune_layer_args(const void* W_in, const void* W_out, const uint8_t* mask_out,
                                       thanos_dtype_t wdtype, int64_t c, int64_t b,
                                       const float* factor, const float* xnorm, thanos_mode_t mode,
                                       double p, int32_t n, int32_t m, int32_t B,
                                       const thanos_stats_t* stats_dev);
thanos_status_t prune_layer_impl(const void* W_in, void* W_out, uint8_t* mask_out,
                                 thanos_dtype_t wdtype, int64_t c, int64_t b, const float* U,
                                 const float* xnorm, thanos_mode_t mode, double p, int32_t n,
                                 int32_t m, int32_t B, void* workspace, size_t ws_bytes,
                                 thanos_stats_t* stats, cudaStream_t stream);
}  // namespace thanos

namespace {

// 4 MiB per GPU that loads the library, held until the process exits.
constexpr size_t kNoAllocScratchBytes = 4u << 20;
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

// In host code `g_noalloc_scratch` is only a handle for the runtime, not a device address; the
// address each device maps it to is looked up once per device and cached here.
constexpr int kMaxDevices = 64;
void* g_scratch_addr[kMaxDevices] = {};
std::mutex g_scratch_mutex;

thanos_status_t scratch_for_current_device(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return THANOS_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (g_scratch_addr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || p == nullptr)
      return THANOS_ERR_CUDA;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return THANOS_OK;
}

}  // namespace

extern "C" thanos_status_t thanos_prune_layer_noalloc(
    const void* W_in, void* W_out, uint8_t* mask_out, thanos_dtype_t wdtype, int64_t c, int64_t b,
    const float* factor, const float* xnorm, thanos_mode_t mode, double p, int32_t n, int32_t m,
    int32_t B, thanos_stats_t* stats_dev, void* stream) {
  using namespace thanos;
  THANOS_TRY(check_prune_layer_args(W_in, W_out, mask_out, wdtype, c, b, factor, xnorm, mode, p, n,
                                    m, B, stats_dev));
  // the layer's scratch must fit the fixed array
  if (prune_workspace_bytes(c, b, B, wdtype) > kNoAllocScratchBytes) return THANOS_ERR_WORKSPACE;
  // The scratch belongs to the CURRENT device; weights that live on another device would be
  // swept with the wrong GPU's array (and launched on the wrong GPU).
  {
    int dev = -1;
    cudaPointerAttributes attr;
    if (cudaGetDevice(&dev) != cudaSuccess) return THANOS_ERR_CUDA;
    if (cudaPointerGetAttributes(&attr, W_in) != cudaSuccess) {
      cudaGetLastError();
      return THANOS_ERR_INVALID_ARG;
    }
    if (attr.type == cudaMemoryTypeDevice && attr.device != dev) return THANOS_ERR_INVALID_ARG;
  }
  void* scratch = nullptr;
  THANOS_TRY(scratch_for_current_device(&scratch));
  // The sweep itself resets what has to start at zero (histogram, sweep state) and writes every
  // other scratch region before reading it, so the previous call's leftovers are harmless.
  return prune_layer_impl(W_in, W_out, mask_out, wdtype, c, b, factor, xnorm, mode, p, n, m, B,
                          scratch, kNoAllocScratchBytes, stats_dev,
                          static_cast<cudaStream_t>(stream));
}
