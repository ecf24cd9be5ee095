// Measurement aid: a kernel of nothing but dependent fp32 FMA chains, to measure the plain-ALU
// (non-tensor) fp32 peak of the device the library runs on.  The per-row solves are bound by
// this pipe, so their roofline fraction needs a measured denominator.
#include "common.cuh"

namespace thanos {
namespace {

constexpr int PROBE_THREADS = 256;
constexpr int PROBE_CHAINS = 16;  // independent accumulators per thread (covers the FMA latency)

__global__ void __launch_bounds__(PROBE_THREADS)
fma_probe_kernel(float* __restrict__ out, int iters, float a, float b) {
  float acc[PROBE_CHAINS];
#pragma unroll
  for (int k = 0; k < PROBE_CHAINS; ++k) acc[k] = (float)(threadIdx.x + k) * 1e-3f;
  for (int it = 0; it < iters; ++it) {
#pragma unroll
    for (int u = 0; u < 4; ++u) {
#pragma unroll
      for (int k = 0; k < PROBE_CHAINS; ++k) acc[k] = fmaf(acc[k], a, b);
    }
  }
  float s = 0.f;
#pragma unroll
  for (int k = 0; k < PROBE_CHAINS; ++k) s += acc[k];
  // one store per thread keeps the chains alive
  out[(size_t)blockIdx.x * PROBE_THREADS + threadIdx.x] = s;
}

}  // namespace
}  // namespace thanos

extern "C" thanos_status_t thanos_fp32_fma_probe(float* out, int64_t out_elems, int32_t ctas,
                                                 int32_t iters, double* flop_out, void* stream) {
  using namespace thanos;
  if (!out || ctas < 1 || iters < 1 || ctas > (1 << 20)) return THANOS_ERR_INVALID_ARG;
  if (out_elems < (int64_t)ctas * PROBE_THREADS) return THANOS_ERR_WORKSPACE;
  if (!aligned16(out)) return THANOS_ERR_ALIGNMENT;
  fma_probe_kernel<<<ctas, PROBE_THREADS, 0, static_cast<cudaStream_t>(stream)>>>(
      out, iters, 0.999f, 1e-4f);
  THANOS_CHECK_LAUNCH();
  if (flop_out)
    *flop_out = 2.0 * (double)ctas * PROBE_THREADS * PROBE_CHAINS * 4.0 * (double)iters;
  return THANOS_OK;
}
