// thanos_hessian_accumulate dispatch: tensor-core path for real layer shapes, plain-ALU path
// for shapes too small to fill one tile.
#include "common.cuh"

namespace thanos {

thanos_status_t hessian_accumulate_simt(float* H, int64_t b, const void* X, thanos_dtype_t xdtype,
                                        int64_t n_tok, int64_t ldx, cudaStream_t stream,
                                        bool ordered);
size_t hessian_tc_workspace_bytes(int64_t b, thanos_dtype_t dtype);
bool hessian_tc_supported(int64_t b, int64_t n_tok);
thanos_status_t hessian_accumulate_tc(float* H, int64_t b, const void* X, thanos_dtype_t xdtype,
                                      int64_t n_tok, int64_t ldx, void* workspace,
                                      cudaStream_t stream, bool ordered);

size_t hessian_workspace_bytes(int64_t b, thanos_dtype_t dtype) {
  return hessian_tc_workspace_bytes(b, dtype);
}

thanos_status_t hessian_accumulate_impl(float* H, int64_t b, const void* X, thanos_dtype_t xdtype,
                                        int64_t n_tok, int64_t ldx, void* workspace,
                                        size_t ws_bytes, cudaStream_t stream, bool ordered) {
  (void)ws_bytes;
  if (hessian_tc_supported(b, n_tok))
    return hessian_accumulate_tc(H, b, X, xdtype, n_tok, ldx, workspace, stream, ordered);
  return hessian_accumulate_simt(H, b, X, xdtype, n_tok, ldx, stream, ordered);
}

}  // namespace thanos
