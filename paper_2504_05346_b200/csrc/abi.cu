// extern "C" entry points: argument checks, workspace carving, dispatch.
#include "common.cuh"
#include "tc_gemm.cuh"

namespace thanos {

std::atomic<long long> g_launch_count{0};

size_t hessian_workspace_bytes(int64_t b, thanos_dtype_t dtype);
thanos_status_t hessian_accumulate_impl(float* H, int64_t b, const void* X, thanos_dtype_t xdtype,
                                        int64_t n_tok, int64_t ldx, void* workspace,
                                        size_t ws_bytes, cudaStream_t stream, bool ordered);
size_t prepare_workspace_bytes(int64_t b);
thanos_status_t prepare_inverse_impl(const float* H, int64_t b, float damp_rel, float* factor,
                                     float* xnorm, void* workspace, size_t ws_bytes,
                                     int32_t* status_dev, cudaStream_t stream);
size_t prune_workspace_bytes(int64_t c, int64_t b, int32_t B, thanos_dtype_t dtype);
size_t prune_outliers_workspace_bytes(int64_t c, int64_t b, int32_t B, thanos_dtype_t dtype);
thanos_status_t prune_layer_outliers_impl(const void* W_in, void* W_out, uint8_t* mask_out,
                                          thanos_dtype_t wdtype, int64_t c, int64_t b,
                                          const float* U, const float* xnorm, const float* H,
                                          int32_t n, int32_t m, int32_t B, double alpha,
                                          uint8_t* row_flags_out, void* workspace, size_t ws_bytes,
                                          thanos_stats_t* stats, cudaStream_t stream);
size_t structured_workspace_bytes(int64_t c, int64_t b, double p, double alpha,
                                  thanos_dtype_t dtype);
thanos_status_t prune_layer_structured_impl(const void* W_in, void* W_out, uint8_t* col_removed_out,
                                            uint8_t* row_outlier_out, thanos_dtype_t wdtype,
                                            int64_t c, int64_t b, const float* U,
                                            const float* xnorm, const float* H, double p,
                                            double alpha, void* workspace, size_t ws_bytes,
                                            thanos_stats_t* stats, cudaStream_t stream);
thanos_status_t validate_sweep_args(int64_t c, int64_t b, thanos_mode_t mode, double p, int32_t n,
                                    int32_t m, int32_t B);
thanos_status_t prune_block_impl(float* Wc, uint8_t* mask, int64_t c, int64_t b, const float* U,
                                 const float* xnorm, thanos_mode_t mode, int32_t n, int32_t m,
                                 int32_t B, int64_t j1, int64_t* r_dev, void* workspace,
                                 size_t ws_bytes, thanos_stats_t* stats, cudaStream_t stream);
thanos_status_t prune_layer_impl(const void* W_in, void* W_out, uint8_t* mask_out,
                                 thanos_dtype_t wdtype, int64_t c, int64_t b, const float* U,
                                 const float* xnorm, thanos_mode_t mode, double p, int32_t n,
                                 int32_t m, int32_t B, void* workspace, size_t ws_bytes,
                                 thanos_stats_t* stats, cudaStream_t stream);

// Host-side argument checks shared by thanos_prune_layer and thanos_prune_layer_noalloc
// (everything except the workspace).
thanos_status_t check_prune_layer_args(const void* W_in, const void* W_out, const uint8_t* mask_out,
                                       thanos_dtype_t wdtype, int64_t c, int64_t b,
                                       const float* factor, const float* xnorm, thanos_mode_t mode,
                                       double p, int32_t n, int32_t m, int32_t B,
                                       const thanos_stats_t* stats_dev) {
  if (!W_in || !W_out || !mask_out || !factor || !xnorm || !stats_dev)
    return THANOS_ERR_INVALID_ARG;
  if (wdtype != THANOS_F32 && wdtype != THANOS_BF16) return THANOS_ERR_DTYPE;
  THANOS_TRY(validate_sweep_args(c, b, mode, p, n, m, B));
  if (!aligned16(W_in) || !aligned16(W_out) || !aligned16(mask_out) || !aligned16(factor) ||
      !aligned16(xnorm) || !aligned16(stats_dev))
    return THANOS_ERR_ALIGNMENT;
  return THANOS_OK;
}

namespace {

// dst keeps the first non-zero status word it is offered
__global__ void fold_word_kernel(int32_t* dst, const int32_t* src) {
  if (*src != 0 && *dst == 0) *dst = *src;
}

constexpr int64_t MAX_B = 65536;
constexpr int64_t HOST_TOKEN_CHUNK = 16384;

size_t elt_size(thanos_dtype_t d) { return d == THANOS_F32 ? 4 : 2; }
bool dtype_ok(thanos_dtype_t d) { return d == THANOS_F32 || d == THANOS_BF16; }

struct HostLayerLayout {
  size_t H, U, xnorm, status, stats, Xstage, Win, Wout, mask, ws, ws_bytes, total;
};

HostLayerLayout host_layout(int64_t c, int64_t b, int32_t B, thanos_dtype_t dtype) {
  HostLayerLayout L;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t o = off;
    off += round_up(bytes, 256);
    return o;
  };
  L.H = take((size_t)b * b * 4);
  L.U = take((size_t)b * b * 4);
  L.xnorm = take((size_t)b * 4);
  L.status = take(16);
  L.stats = take(sizeof(thanos_stats_t));
  L.Xstage = take(2 * (size_t)HOST_TOKEN_CHUNK * b * elt_size(dtype));
  L.Win = take((size_t)c * b * elt_size(dtype));
  L.Wout = take((size_t)c * b * elt_size(dtype));
  L.mask = take((size_t)c * b);
  size_t w = hessian_workspace_bytes(b, dtype);
  size_t w2 = prepare_workspace_bytes(b);
  size_t w3 = prune_workspace_bytes(c, b, B, dtype);
  L.ws_bytes = w > w2 ? w : w2;
  if (w3 > L.ws_bytes) L.ws_bytes = w3;
  L.ws = take(L.ws_bytes);
  L.total = off;
  return L;
}

}  // namespace
}  // namespace thanos

using namespace thanos;

extern "C" {

static thanos_status_t hessian_accumulate_checked(float* H, int64_t b, const void* X,
                                                  thanos_dtype_t xdtype, int64_t n_tok, int64_t ldx,
                                                  void* workspace, size_t ws_bytes, void* stream,
                                                  bool ordered) {
  if (!H || (!X && n_tok > 0)) return THANOS_ERR_INVALID_ARG;
  if (!dtype_ok(xdtype)) return THANOS_ERR_DTYPE;
  if (b < 8 || b > MAX_B || b % 8 != 0 || n_tok < 0) return THANOS_ERR_SHAPE;
  if (ldx < b || ldx % 8 != 0) return THANOS_ERR_ALIGNMENT;
  if (!aligned16(H) || !aligned16(X) || !aligned16(workspace)) return THANOS_ERR_ALIGNMENT;
  if (n_tok == 0) return THANOS_OK;
  if (ws_bytes < hessian_workspace_bytes(b, xdtype) || (!workspace && ws_bytes > 0))
    return THANOS_ERR_WORKSPACE;
  return hessian_accumulate_impl(H, b, X, xdtype, n_tok, ldx, workspace, ws_bytes,
                                 static_cast<cudaStream_t>(stream), ordered);
}

thanos_status_t thanos_hessian_accumulate(float* H, int64_t b, const void* X, thanos_dtype_t xdtype,
                                          int64_t n_tok, int64_t ldx, void* workspace,
                                          size_t ws_bytes, void* stream) {
  return hessian_accumulate_checked(H, b, X, xdtype, n_tok, ldx, workspace, ws_bytes, stream, false);
}

thanos_status_t thanos_hessian_accumulate_ordered(float* H, int64_t b, const void* X,
                                                  thanos_dtype_t xdtype, int64_t n_tok, int64_t ldx,
                                                  void* workspace, size_t ws_bytes, void* stream) {
  return hessian_accumulate_checked(H, b, X, xdtype, n_tok, ldx, workspace, ws_bytes, stream, true);
}

thanos_status_t thanos_prepare_inverse(const float* H, int64_t b, float damp_rel, float* factor,
                                       float* xnorm, void* workspace, size_t ws_bytes,
                                       int32_t* status_dev, void* stream) {
  if (!H || !factor || !xnorm || !status_dev) return THANOS_ERR_INVALID_ARG;
  if (!(damp_rel >= 0.f)) return THANOS_ERR_INVALID_ARG;
  if (b < 8 || b > MAX_B || b % 8 != 0) return THANOS_ERR_SHAPE;
  if (!aligned16(H) || !aligned16(factor) || !aligned16(xnorm) || !aligned16(workspace))
    return THANOS_ERR_ALIGNMENT;
  if (!workspace || ws_bytes < prepare_workspace_bytes(b)) return THANOS_ERR_WORKSPACE;
  return prepare_inverse_impl(H, b, damp_rel, factor, xnorm, workspace, ws_bytes, status_dev,
                              static_cast<cudaStream_t>(stream));
}

thanos_status_t thanos_prune_layer(const void* W_in, void* W_out, uint8_t* mask_out,
                                   thanos_dtype_t wdtype, int64_t c, int64_t b,
                                   const float* factor, const float* xnorm, thanos_mode_t mode,
                                   double p, int32_t n, int32_t m, int32_t B, void* workspace,
                                   size_t ws_bytes, thanos_stats_t* stats_dev, void* stream) {
  THANOS_TRY(check_prune_layer_args(W_in, W_out, mask_out, wdtype, c, b, factor, xnorm, mode, p, n,
                                    m, B, stats_dev));
  if (!aligned16(workspace)) return THANOS_ERR_ALIGNMENT;
  if (!workspace || ws_bytes < prune_workspace_bytes(c, b, B, wdtype)) return THANOS_ERR_WORKSPACE;
  return prune_layer_impl(W_in, W_out, mask_out, wdtype, c, b, factor, xnorm, mode, p, n, m, B,
                          workspace, ws_bytes, stats_dev, static_cast<cudaStream_t>(stream));
}

thanos_status_t thanos_prune_layer_outliers(const void* W_in, void* W_out, uint8_t* mask_out,
                                            thanos_dtype_t wdtype, int64_t c, int64_t b,
                                            const float* factor, const float* xnorm,
                                            const float* H, int32_t n, int32_t m, int32_t B,
                                            double alpha, uint8_t* row_outlier_out,
                                            void* workspace, size_t ws_bytes,
                                            thanos_stats_t* stats_dev, void* stream) {
  if (!W_in || !W_out || !mask_out || !factor || !xnorm || !H || !stats_dev)
    return THANOS_ERR_INVALID_ARG;
  if (!dtype_ok(wdtype)) return THANOS_ERR_DTYPE;
  if (!(alpha >= 0.0 && alpha < 1.0)) return THANOS_ERR_INVALID_ARG;
  THANOS_TRY(validate_sweep_args(c, b, THANOS_NM, 0.0, n, m, B));
  if (c > (1 << 24)) return THANOS_ERR_SHAPE;
  if (!aligned16(W_in) || !aligned16(W_out) || !aligned16(mask_out) || !aligned16(factor) ||
      !aligned16(xnorm) || !aligned16(H) || !aligned16(workspace) || !aligned16(stats_dev))
    return THANOS_ERR_ALIGNMENT;
  if (!workspace || ws_bytes < prune_outliers_workspace_bytes(c, b, B, wdtype))
    return THANOS_ERR_WORKSPACE;
  return prune_layer_outliers_impl(W_in, W_out, mask_out, wdtype, c, b, factor, xnorm, H, n, m, B,
                                   alpha, row_outlier_out, workspace, ws_bytes, stats_dev,
                                   static_cast<cudaStream_t>(stream));
}

thanos_status_t thanos_prune_layer_structured(const void* W_in, void* W_out,
                                              uint8_t* col_removed_out, uint8_t* row_outlier_out,
                                              thanos_dtype_t wdtype, int64_t c, int64_t b,
                                              const float* factor, const float* xnorm,
                                              const float* H, double p, double alpha,
                                              void* workspace, size_t ws_bytes,
                                              thanos_stats_t* stats_dev, void* stream) {
  if (!W_in || !W_out || !factor || !xnorm || !stats_dev) return THANOS_ERR_INVALID_ARG;
  if (!dtype_ok(wdtype)) return THANOS_ERR_DTYPE;
  if (!(alpha >= 0.0 && alpha < 1.0) || !(p >= 0.0 && p < 1.0)) return THANOS_ERR_INVALID_ARG;
  if (alpha > 0.0 && !H) return THANOS_ERR_INVALID_ARG;
  if (c < 1 || c > (1 << 24) || b < 8 || b > MAX_B || b % 8 != 0) return THANOS_ERR_SHAPE;
  if (!aligned16(W_in) || !aligned16(W_out) || !aligned16(factor) || !aligned16(xnorm) ||
      !aligned16(H) || !aligned16(workspace) || !aligned16(stats_dev))
    return THANOS_ERR_ALIGNMENT;
  const size_t need = structured_workspace_bytes(c, b, p, alpha, wdtype);
  if (need == 0) return THANOS_ERR_INVALID_ARG;  // p / (1 - alpha) leaves no column
  if (!workspace || ws_bytes < need) return THANOS_ERR_WORKSPACE;
  return prune_layer_structured_impl(W_in, W_out, col_removed_out, row_outlier_out, wdtype, c, b,
                                     factor, xnorm, H, p, alpha, workspace, ws_bytes, stats_dev,
                                     static_cast<cudaStream_t>(stream));
}

size_t thanos_structured_workspace_bytes(int64_t c, int64_t b, double p, double alpha,
                                         thanos_dtype_t dtype) {
  if (c < 1 || b < 8 || b > MAX_B || b % 8 != 0 || !dtype_ok(dtype)) return 0;
  if (!(alpha >= 0.0 && alpha < 1.0) || !(p >= 0.0 && p < 1.0)) return 0;
  return structured_workspace_bytes(c, b, p, alpha, dtype);
}

thanos_status_t thanos_prune_block(float* Wc, uint8_t* mask, int64_t c, int64_t b,
                                   const float* factor, const float* xnorm, thanos_mode_t mode,
                                   int32_t n, int32_t m, int32_t B, int64_t j1, int64_t* r_dev,
                                   void* workspace, size_t ws_bytes, thanos_stats_t* stats_dev,
                                   void* stream) {
  if (!Wc || !mask || !factor || !xnorm || !stats_dev) return THANOS_ERR_INVALID_ARG;
  if (mode == THANOS_UNSTRUCTURED && !r_dev) return THANOS_ERR_INVALID_ARG;
  THANOS_TRY(validate_sweep_args(c, b, mode, 0.0, n, m, B));
  if (j1 < 0 || j1 >= b || j1 % B != 0) return THANOS_ERR_SHAPE;
  if (!aligned16(Wc) || !aligned16(mask) || !aligned16(factor) || !aligned16(xnorm) ||
      !aligned16(workspace) || !aligned16(stats_dev))
    return THANOS_ERR_ALIGNMENT;
  if (!workspace || ws_bytes < prune_workspace_bytes(c, b, B, THANOS_F32))
    return THANOS_ERR_WORKSPACE;
  return prune_block_impl(Wc, mask, c, b, factor, xnorm, mode, n, m, B, j1, r_dev, workspace,
                          ws_bytes, stats_dev, static_cast<cudaStream_t>(stream));
}

thanos_status_t thanos_prune_layer_host(const void* W_in_host, const void* X_host,
                                        void* W_out_host, uint8_t* mask_out_host,
                                        thanos_dtype_t dtype, int64_t c, int64_t b, int64_t a,
                                        float damp_rel, thanos_mode_t mode, double p, int32_t n,
                                        int32_t m, int32_t B, int32_t reuse_factor, void* arena,
                                        size_t arena_bytes, thanos_stats_t* stats_host,
                                        void* stream_v) {
  if (!W_in_host || !W_out_host || !mask_out_host || !arena || !stats_host)
    return THANOS_ERR_INVALID_ARG;
  if (!reuse_factor && (!X_host || a < 1)) return THANOS_ERR_INVALID_ARG;
  if (!dtype_ok(dtype)) return THANOS_ERR_DTYPE;
  if (!(damp_rel >= 0.f)) return THANOS_ERR_INVALID_ARG;
  if (b < 8 || b > MAX_B || b % 8 != 0) return THANOS_ERR_SHAPE;
  THANOS_TRY(validate_sweep_args(c, b, mode, p, n, m, B));
  if (!aligned16(arena)) return THANOS_ERR_ALIGNMENT;
  HostLayerLayout L = host_layout(c, b, B, dtype);
  if (arena_bytes < L.total) return THANOS_ERR_WORKSPACE;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  char* base = static_cast<char*>(arena);
  float* H = reinterpret_cast<float*>(base + L.H);
  float* U = reinterpret_cast<float*>(base + L.U);
  float* xnorm = reinterpret_cast<float*>(base + L.xnorm);
  int32_t* status = reinterpret_cast<int32_t*>(base + L.status);
  thanos_stats_t* stats = reinterpret_cast<thanos_stats_t*>(base + L.stats);
  void* ws = base + L.ws;
  const size_t es = elt_size(dtype);

  THANOS_CUDA(cudaMemcpyAsync(base + L.Win, W_in_host, (size_t)c * b * es, cudaMemcpyHostToDevice,
                              stream));
  if (!reuse_factor) {
    THANOS_CUDA(cudaMemsetAsync(H, 0, (size_t)b * b * 4, stream));
    THANOS_CUDA(cudaMemsetAsync(status, 0, 16, stream));
    // Two staging buffers: the copy of chunk k+1 is issued on a second stream while chunk k is
    // being accumulated.
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t evs[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};
    thanos_status_t st = THANOS_OK;
    if (cudaStreamCreateWithFlags(&copy_stream, cudaStreamNonBlocking) != cudaSuccess)
      st = THANOS_ERR_CUDA;
    for (int i = 0; i < 5 && st == THANOS_OK; ++i)
      if (cudaEventCreateWithFlags(&evs[i], cudaEventDisableTiming) != cudaSuccess)
        st = THANOS_ERR_CUDA;
    cudaEvent_t* copied = evs;        // [2]
    cudaEvent_t* consumed = evs + 2;  // [2]
    cudaEvent_t start = evs[4];
    if (st == THANOS_OK && (cudaEventRecord(start, stream) != cudaSuccess ||
                            cudaStreamWaitEvent(copy_stream, start, 0) != cudaSuccess))
      st = THANOS_ERR_CUDA;
    int64_t k = 0;
    for (int64_t t0 = 0; t0 < a && st == THANOS_OK; t0 += HOST_TOKEN_CHUNK, ++k) {
      int64_t nt = a - t0 < HOST_TOKEN_CHUNK ? a - t0 : HOST_TOKEN_CHUNK;
      int slot = (int)(k & 1);
      char* stage = base + L.Xstage + (size_t)slot * HOST_TOKEN_CHUNK * b * es;
      bool ok = true;
      if (k >= 2) ok = cudaStreamWaitEvent(copy_stream, consumed[slot], 0) == cudaSuccess;
      ok = ok && cudaMemcpyAsync(stage, static_cast<const char*>(X_host) + (size_t)t0 * b * es,
                                 (size_t)nt * b * es, cudaMemcpyHostToDevice,
                                 copy_stream) == cudaSuccess;
      ok = ok && cudaEventRecord(copied[slot], copy_stream) == cudaSuccess;
      ok = ok && cudaStreamWaitEvent(stream, copied[slot], 0) == cudaSuccess;
      if (!ok) {
        st = THANOS_ERR_CUDA;
        break;
      }
      st = thanos_hessian_accumulate(H, b, stage, dtype, nt, b, ws, L.ws_bytes, stream);
      if (st == THANOS_OK) {
        // the accumulation's own status word (first word of its workspace) is cleared by the next
        // chunk and overwritten by the later calls: keep the first failure in status[2]
        fold_word_kernel<<<1, 1, 0, stream>>>(status + 2, static_cast<const int32_t*>(ws));
        count_launch();
        if (cudaGetLastError() != cudaSuccess) st = THANOS_ERR_CUDA;
      }
      if (cudaEventRecord(consumed[slot], stream) != cudaSuccess && st == THANOS_OK)
        st = THANOS_ERR_CUDA;
    }
    // the staging buffers and the temporary stream / events are released only when every copy
    // issued above has finished
    if (copy_stream) {
      cudaStreamSynchronize(copy_stream);
      cudaStreamDestroy(copy_stream);
    }
    for (int i = 0; i < 5; ++i)
      if (evs[i]) cudaEventDestroy(evs[i]);
    THANOS_TRY(st);
    THANOS_TRY(thanos_prepare_inverse(H, b, damp_rel, U, xnorm, ws, L.ws_bytes, status, stream));
  }
  THANOS_TRY(thanos_prune_layer(base + L.Win, base + L.Wout, reinterpret_cast<uint8_t*>(base + L.mask),
                                dtype, c, b, U, xnorm, mode, p, n, m, B, ws, L.ws_bytes, stats,
                                stream));
  THANOS_CUDA(cudaMemcpyAsync(W_out_host, base + L.Wout, (size_t)c * b * es, cudaMemcpyDeviceToHost,
                              stream));
  THANOS_CUDA(cudaMemcpyAsync(mask_out_host, base + L.mask, (size_t)c * b, cudaMemcpyDeviceToHost,
                              stream));
  THANOS_CUDA(cudaMemcpyAsync(stats_host, stats, sizeof(thanos_stats_t), cudaMemcpyDeviceToHost,
                              stream));
  int32_t st_host[4] = {0, 0, 0, 0};
  THANOS_CUDA(cudaMemcpyAsync(st_host, status, 16, cudaMemcpyDeviceToHost, stream));
  THANOS_CUDA(cudaStreamSynchronize(stream));
  if (st_host[2] != 0 && stats_host->status == 0) {  // Hessian accumulation (bounded wait ran out)
    stats_host->status = st_host[2];
    stats_host->err_index = -1;
  }
  if (st_host[0] != 0 && stats_host->status == 0) {  // factorisation
    stats_host->status = st_host[0];
    stats_host->err_index = st_host[1];
  }
  return THANOS_OK;
}

size_t thanos_dense_product_workspace(int64_t M, int64_t N, int64_t K) {
  if (M < 1 || N < 1 || K < 1) return 0;
  const size_t Kp = round_up((size_t)K, 8), Np = round_up((size_t)N, 8);
  const size_t a = round_up(3 * (size_t)M * Kp * 2, 256);
  const size_t bt = 3 * (size_t)N * Kp * 2, bn = 3 * (size_t)K * Np * 2;
  return 256 + a + round_up(bt > bn ? bt : bn, 256);
}

thanos_status_t thanos_dense_product(float* D, int64_t ldd, const float* A, int64_t lda,
                                     const float* B, int64_t ldb, int32_t b_transposed, int64_t M,
                                     int64_t N, int64_t K, float alpha, int32_t accumulate,
                                     void* workspace, size_t ws_bytes, void* stream_v) {
  if (!D || !A || !B || !workspace) return THANOS_ERR_INVALID_ARG;
  if (M < 1 || N < 1 || K < 1 || M > (1 << 30) || N > (1 << 30) || K > (1 << 30))
    return THANOS_ERR_SHAPE;
  if (ldd % 4 || lda % 4 || ldb % 4 || K % 4 || (!b_transposed && N % 4)) return THANOS_ERR_ALIGNMENT;
  if (ldd < N || lda < K || ldb < (b_transposed ? K : N)) return THANOS_ERR_SHAPE;
  if (!aligned16(D) || !aligned16(A) || !aligned16(B) || !aligned16(workspace))
    return THANOS_ERR_ALIGNMENT;
  if (ws_bytes < thanos_dense_product_workspace(M, N, K)) return THANOS_ERR_WORKSPACE;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  const int64_t Kp = (int64_t)round_up((size_t)K, 8), Np = (int64_t)round_up((size_t)N, 8);
  char* base = static_cast<char*>(workspace);
  int32_t* status = reinterpret_cast<int32_t*>(base);
  __nv_bfloat16* Ap = reinterpret_cast<__nv_bfloat16*>(base + 256);
  __nv_bfloat16* Bp =
      reinterpret_cast<__nv_bfloat16*>(base + 256 + round_up(3 * (size_t)M * Kp * 2, 256));
  THANOS_CUDA(cudaMemsetAsync(status, 0, 16, stream));
  THANOS_TRY(split3_planes(A, lda, M, K, Ap, Kp, M * Kp, stream));
  TcGemmArgs g;
  if (b_transposed) {
    THANOS_TRY(split3_planes(B, ldb, N, K, Bp, Kp, N * Kp, stream));
    g.ldb = Kp;
    g.b_plane = N * Kp;
  } else {
    THANOS_TRY(split3_planes(B, ldb, K, N, Bp, Np, K * Np, stream));
    g.ldb = Np;
    g.b_plane = K * Np;
  }
  g.D = D;
  g.ldd = ldd;
  g.A = Ap;
  g.lda = Kp;
  g.a_plane = M * Kp;
  g.B = Bp;
  g.b_kmajor = b_transposed ? 1 : 0;
  g.M = (int)M;
  g.N = (int)N;
  g.K = (int)K;
  g.alpha = alpha;
  g.accumulate = accumulate ? 1 : 0;
  g.status = status;
  return tc_gemm_split3(g, stream);
}

size_t thanos_workspace_bytes(int32_t which, int64_t c, int64_t b, int32_t B, thanos_dtype_t dtype) {
  if (b < 8 || b > MAX_B || b % 8 != 0 || !dtype_ok(dtype)) return 0;
  switch (which) {
    case THANOS_WS_HESSIAN:
      return hessian_workspace_bytes(b, dtype);
    case THANOS_WS_PREPARE:
      return prepare_workspace_bytes(b);
    case THANOS_WS_PRUNE:
      if (c < 1 || B < 1 || B > 512) return 0;
      return prune_workspace_bytes(c, b, B, dtype);
    case THANOS_WS_PRUNE_OUTLIERS:
      if (c < 1 || B < 1 || B > 512) return 0;
      return prune_outliers_workspace_bytes(c, b, B, dtype);
    case THANOS_WS_HOST_LAYER:
      if (c < 1 || B < 1 || B > 512) return 0;
      return host_layout(c, b, B, dtype).total;
    default:
      return 0;
  }
}

const char* thanos_status_string(thanos_status_t status) {
  switch (status) {
    case THANOS_OK: return "ok";
    case THANOS_ERR_INVALID_ARG: return "invalid argument";
    case THANOS_ERR_SHAPE: return "unsupported shape";
    case THANOS_ERR_DTYPE: return "unsupported dtype";
    case THANOS_ERR_ALIGNMENT: return "misaligned pointer or leading dimension";
    case THANOS_ERR_WORKSPACE: return "workspace missing or too small";
    case THANOS_ERR_NOT_SPD: return "matrix not positive definite";
    case THANOS_ERR_TIMEOUT: return "device-side wait timed out";
    case THANOS_ERR_CUDA: return "CUDA call failed";
    default: return "unknown status";
  }
}

int32_t thanos_version(void) { return 100; }

int64_t thanos_launch_count(void) { return (int64_t)g_launch_count.load(); }

}  // extern "C"
