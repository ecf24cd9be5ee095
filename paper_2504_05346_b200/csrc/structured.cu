// Structured pruning (Algorithm 2): whole columns are removed, one shared system for all rows.
//
// With q the s = ceil(p b / (1 - alpha)) columns of smallest loss v_j = ||W_{rows, j}||^2 ||X_j||^2
// (rows = all but the ceil(alpha c) outlier rows), every pruned row gets (Eq. 8 with the same q)
//     W <- W - W[:, q] inv(Hinv[q, q]) Hinv[q, :],        W[:, q] <- 0.
// No column or row is physically permuted: the permutations of the listing only bring q and the
// pruned rows to the front, so gathering by index is the same computation.  With U from
// thanos_prepare_inverse (Hinv = U^T U):
//     R     = Hinv[q, :]   = (U[:, q])^T U                       (tensor-core product, s x b)
//     Rhat  = R[:, q]                                             (s x s, SPD)
//     Rhat^{-1} = Ur^T Ur  by the same factorisation as the layer's Hessian
//     Y     = Ur^T (Ur R)                                         (two products, s x b)
//     W    -= W[:, q] Y                                           (one product, c x b)
// All products run on the tensor cores with fp32 operands as three bf16 planes.
#include "common.cuh"
#include "tc_gemm.cuh"

namespace thanos {

size_t outlier_extra_bytes(int64_t c, int64_t b);
thanos_status_t outlier_row_flags(const float* Wc, const float* H, int64_t c, int64_t b, int n_out,
                                  void* scratch, size_t scratch_bytes, uint8_t** flags_dev,
                                  int32_t* tc_status, cudaStream_t stream);
size_t prepare_workspace_bytes(int64_t b);
thanos_status_t convert_to_f32(const __nv_bfloat16* in, float* out, int64_t n, cudaStream_t stream);
thanos_status_t convert_to_bf16(const float* in, __nv_bfloat16* out, int64_t n, cudaStream_t stream);
thanos_status_t prepare_inverse_impl(const float* H, int64_t b, float damp_rel, float* factor,
                                     float* xnorm, void* workspace, size_t ws_bytes,
                                     int32_t* status_dev, cudaStream_t stream);

namespace {

constexpr int ROW_CHUNK = 64;  // rows per partial sum of the column losses

// partial[chunk][j] = sum over the pruned rows of the chunk of W_ij^2 (fixed order: the column
// ranking must not depend on the launch)
__global__ void __launch_bounds__(256)
col_sq_partial_kernel(const float* __restrict__ Wc, const uint8_t* __restrict__ flags, int c, int b,
                      double* __restrict__ partial) {
  const int j = blockIdx.y * 256 + threadIdx.x;
  if (j >= b) return;
  const int r0 = blockIdx.x * ROW_CHUNK;
  const int r1 = min(r0 + ROW_CHUNK, c);
  double acc = 0.0;
  for (int i = r0; i < r1; ++i) {
    if (flags[i]) continue;
    const float w = Wc[(int64_t)i * b + j];
    acc += (double)w * (double)w;
  }
  partial[(int64_t)blockIdx.x * b + j] = acc;
}

// v_j = ||W_{rows, j}||^2 ||X_j||^2
__global__ void __launch_bounds__(256)
col_loss_kernel(const double* __restrict__ partial, int n_chunks, const float* __restrict__ xnorm,
                int b, double* __restrict__ v) {
  const int j = blockIdx.x * 256 + threadIdx.x;
  if (j >= b) return;
  double acc = 0.0;
  for (int k = 0; k < n_chunks; ++k) acc += partial[(int64_t)k * b + j];
  const double xn = (double)xnorm[j];
  v[j] = acc * xn * xn;
}

// exclusive prefix sum of one value per thread over a 1024-thread CTA; *total = sum
__device__ __forceinline__ unsigned block_exclusive_scan(unsigned x, unsigned* warp_sums,
                                                         unsigned* total) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  unsigned incl = x;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += y;
  }
  __syncthreads();  // warp_sums may still be read from an earlier call
  if (lane == 31) warp_sums[wid] = incl;
  __syncthreads();
  if (wid == 0) {
    const unsigned w = warp_sums[lane];
    unsigned wi = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned y = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += y;
    }
    warp_sums[lane] = wi - w;
    if (lane == 31) *total = wi;
  }
  __syncthreads();
  return warp_sums[wid] + incl - x;
}

// The s columns with the smallest v (order (v, column): of equal losses the lower column goes
// first) get colrm = 1; qlist holds them in ascending column order, padded with -1 up to s_pad.
// One CTA: radix select over the 64-bit patterns of the non-negative doubles, then two scans.
__global__ void __launch_bounds__(1024)
smallest_cols_kernel(const double* __restrict__ v, int b, int s, int s_pad,
                     uint8_t* __restrict__ colrm, int* __restrict__ qlist) {
  __shared__ unsigned hist[256];
  __shared__ unsigned long long s_prefix;
  __shared__ unsigned s_k, s_total;
  __shared__ unsigned warp_sums[32];
  const int tid = threadIdx.x;
  for (int a = tid; a < s_pad; a += 1024) qlist[a] = -1;
  if (s <= 0) {
    for (int j = tid; j < b; j += 1024) colrm[j] = 0;
    return;
  }
  if (tid == 0) {
    s_prefix = 0ull;
    s_k = (unsigned)s;  // rank from the bottom still to resolve
  }
  for (int pass = 0; pass < 8; ++pass) {
    const int shift = 56 - 8 * pass;
    if (tid < 256) hist[tid] = 0;
    __syncthreads();
    const unsigned long long prefix = s_prefix;
    for (int j = tid; j < b; j += 1024) {
      const unsigned long long key = (unsigned long long)__double_as_longlong(v[j]);
      if (pass == 0 || (key >> (shift + 8)) == prefix)
        atomicAdd(&hist[(unsigned)(key >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (tid == 0) {
      unsigned k = s_k, bin = 0;
      for (; bin < 255; ++bin) {  // from the smallest digit up
        if (hist[bin] >= k) break;
        k -= hist[bin];
      }
      s_prefix = (prefix << 8) | bin;
      s_k = k;
    }
    __syncthreads();
  }
  const unsigned long long tau = s_prefix;  // pattern of the s-th smallest loss
  // contiguous chunk of columns per thread, so that scans run in column order
  const int per = (b + 1023) / 1024;
  const int j0 = min(tid * per, b), j1 = min(j0 + per, b);
  unsigned lt = 0, eq = 0;
  for (int j = j0; j < j1; ++j) {
    const unsigned long long key = (unsigned long long)__double_as_longlong(v[j]);
    lt += key < tau;
    eq += key == tau;
  }
  const unsigned eq_before = block_exclusive_scan(eq, warp_sums, &s_total);
  (void)block_exclusive_scan(lt, warp_sums, &s_total);
  const unsigned need_eq = (unsigned)s - s_total;  // ties taken, lowest columns first
  unsigned mine = 0, e = eq_before;
  for (int j = j0; j < j1; ++j) {
    const unsigned long long key = (unsigned long long)__double_as_longlong(v[j]);
    const bool rm = key < tau || (key == tau && e < need_eq);
    e += key == tau;
    colrm[j] = rm ? 1 : 0;
    mine += rm;
  }
  unsigned pos = block_exclusive_scan(mine, warp_sums, &s_total);
  for (int j = j0; j < j1; ++j)
    if (colrm[j]) qlist[pos++] = j;
}

// UqT[a][k] = U[k][q_a] as three bf16 planes [s_pad, b] (rows a >= s are zero)
__global__ void __launch_bounds__(256)
gather_uq_kernel(const float* __restrict__ U, int b, const int* __restrict__ qlist, int s_pad,
                 __nv_bfloat16* __restrict__ planes) {
  __shared__ float tile[32][33];
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int k0 = blockIdx.x * 32, a0 = blockIdx.y * 32;
  const int a = a0 + tx;
  const int q = a < s_pad ? qlist[a] : -1;
  for (int i = ty; i < 32; i += 8) {
    const int k = k0 + i;
    tile[i][tx] = (q >= 0 && k < b) ? U[(int64_t)k * b + q] : 0.f;
  }
  __syncthreads();
  const int k = k0 + tx;
  if (k >= b) return;
  for (int i = ty; i < 32; i += 8) {
    const int aa = a0 + i;
    if (aa < s_pad) store_split3(planes + (int64_t)aa * b + k, (int64_t)s_pad * b, tile[tx][i]);
  }
}

// Rhat[a][a2] = R[a][q_a2] (= Hinv[q_a, q_a2]); identity on the padding
__global__ void __launch_bounds__(256)
gather_rhat_kernel(const float* __restrict__ R, int b, const int* __restrict__ qlist, int s_pad,
                   float* __restrict__ Rhat) {
  const int a2 = blockIdx.y * 256 + threadIdx.x;
  const int a = blockIdx.x;
  if (a2 >= s_pad) return;
  const int qa = qlist[a], q2 = qlist[a2];
  float val;
  if (qa >= 0 && q2 >= 0)
    val = R[(int64_t)a * b + q2];
  else
    val = a == a2 ? 1.f : 0.f;
  Rhat[(int64_t)a * s_pad + a2] = val;
}

// planes of the transpose of a square fp32 matrix
__global__ void __launch_bounds__(256)
transpose_split_kernel(const float* __restrict__ in, int n, __nv_bfloat16* __restrict__ planes) {
  __shared__ float tile[32][33];
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
  for (int i = ty; i < 32; i += 8) {
    const int r = r0 + i, cc = c0 + tx;
    tile[i][tx] = (r < n && cc < n) ? in[(int64_t)r * n + cc] : 0.f;
  }
  __syncthreads();
  for (int i = ty; i < 32; i += 8) {
    const int orow = c0 + i, ocol = r0 + tx;  // out[orow][ocol] = in[ocol][orow]
    if (orow < n && ocol < n)
      store_split3(planes + (int64_t)orow * n + ocol, (int64_t)n * n, tile[tx][i]);
  }
}

// Wq[i][a] = W[i][q_a] for the pruned rows (zero for outlier rows and padding), as planes [c, s_pad]
__global__ void __launch_bounds__(256)
gather_wq_kernel(const float* __restrict__ Wc, const uint8_t* __restrict__ flags, int c, int b,
                 const int* __restrict__ qlist, int s_pad, __nv_bfloat16* __restrict__ planes) {
  const int a = blockIdx.y * 256 + threadIdx.x;
  const int i = blockIdx.x;
  if (a >= s_pad) return;
  const int q = qlist[a];
  const float val = (q >= 0 && !flags[i]) ? Wc[(int64_t)i * b + q] : 0.f;
  store_split3(planes + (int64_t)i * s_pad + a, (int64_t)c * s_pad, val);
}

// exact zeros in the removed columns of the pruned rows
__global__ void __launch_bounds__(256)
zero_removed_kernel(float* __restrict__ Wc, const uint8_t* __restrict__ flags,
                    const uint8_t* __restrict__ colrm, int c, int b) {
  const int j = blockIdx.y * 256 + threadIdx.x;
  const int i = blockIdx.x;
  if (j >= b || flags[i] || !colrm[j]) return;
  Wc[(int64_t)i * b + j] = 0.f;
}

__global__ void finish_kernel(thanos_stats_t* stats, const int32_t* prep_status,
                              const int32_t* tc_status, long long n_pruned, int s) {
  thanos_stats_t z = {};
  if (prep_status[0] != 0) {
    z.status = prep_status[0];
    z.err_index = prep_status[1];
  } else if (tc_status[0] != 0) {
    z.status = tc_status[0];
  }
  z.n_pruned = n_pruned;
  z.max_s = s;
  z.n_blocks = 1;
  *stats = z;
}

struct StructWs {
  float* Wc;
  uint8_t* flags;
  uint8_t* colrm;
  int* qlist;
  double* partial;
  double* v;
  __nv_bfloat16* UqT;  // [3][s_pad, b]
  __nv_bfloat16* Up;   // [3][b, b]
  float* R;            // [s_pad, b]
  __nv_bfloat16* Rp;   // [3][s_pad, b]
  float* Rhat;         // [s_pad, s_pad]
  float* Ur;           // [s_pad, s_pad]
  float* xdummy;       // [s_pad]
  __nv_bfloat16* Urp;  // [3][s_pad, s_pad]
  __nv_bfloat16* UrTp; // [3][s_pad, s_pad]
  __nv_bfloat16* Zp;   // [3][s_pad, b]
  __nv_bfloat16* Yp;   // [3][s_pad, b]
  __nv_bfloat16* Wqp;  // [3][c, s_pad]
  int32_t* status;     // [0..1] factorisation, [4..] tensor-core products
  void* prep;
  size_t prep_bytes;
  void* outl;
  size_t outl_bytes;
};

int64_t padded(int64_t s) { return s < 8 ? 8 : (s + 7) / 8 * 8; }

bool carve_struct(StructWs& w, void* ws, size_t ws_bytes, int64_t c, int64_t b, int64_t sp,
                  bool need_wc, bool need_outl) {
  Arena ar(ws, ws_bytes);
  const size_t chunks = (size_t)ceil_div(c, ROW_CHUNK);
  w.Wc = need_wc ? ar.take<float>((size_t)c * b) : nullptr;
  w.flags = ar.take<uint8_t>((size_t)c);
  w.colrm = ar.take<uint8_t>((size_t)b);
  w.qlist = ar.take<int>((size_t)sp);
  w.partial = ar.take<double>(chunks * (size_t)b);
  w.v = ar.take<double>((size_t)b);
  w.UqT = ar.take<__nv_bfloat16>(3 * (size_t)sp * b);
  w.Up = ar.take<__nv_bfloat16>(3 * (size_t)b * b);
  w.R = ar.take<float>((size_t)sp * b);
  w.Rp = ar.take<__nv_bfloat16>(3 * (size_t)sp * b);
  w.Rhat = ar.take<float>((size_t)sp * sp);
  w.Ur = ar.take<float>((size_t)sp * sp);
  w.xdummy = ar.take<float>((size_t)sp);
  w.Urp = ar.take<__nv_bfloat16>(3 * (size_t)sp * sp);
  w.UrTp = ar.take<__nv_bfloat16>(3 * (size_t)sp * sp);
  w.Zp = ar.take<__nv_bfloat16>(3 * (size_t)sp * b);
  w.Yp = ar.take<__nv_bfloat16>(3 * (size_t)sp * b);
  w.Wqp = ar.take<__nv_bfloat16>(3 * (size_t)c * sp);
  w.status = ar.take<int32_t>(16);
  w.prep_bytes = prepare_workspace_bytes(sp);
  w.prep = ar.take<char>(w.prep_bytes);
  w.outl_bytes = need_outl ? outlier_extra_bytes(c, b) : 0;
  w.outl = need_outl ? ar.take<char>(w.outl_bytes) : nullptr;
  return ar.ok();
}

}  // namespace

int64_t structured_column_count(double p, int64_t b, double alpha) {
  return (int64_t)ceil(p * (double)b / (1.0 - alpha) - 1e-12);
}

size_t structured_workspace_bytes(int64_t c, int64_t b, double p, double alpha,
                                  thanos_dtype_t dtype) {
  const int64_t s = structured_column_count(p, b, alpha);
  if (s < 0 || s >= b) return 0;
  const size_t sp = (size_t)padded(s);
  const size_t chunks = (size_t)ceil_div(c, ROW_CHUNK);
  auto r = [](size_t x) { return round_up(x, 256); };
  size_t t = dtype != THANOS_F32 ? r((size_t)c * b * 4) : 0;
  t += r((size_t)c) + r((size_t)b) + r(sp * 4) + r(chunks * (size_t)b * 8) + r((size_t)b * 8);
  t += 4 * r(3 * sp * (size_t)b * 2);                  // UqT, Rp, Zp, Yp
  t += r(3 * (size_t)b * b * 2);                       // Up
  t += r(sp * (size_t)b * 4) + 2 * r(sp * sp * 4) + r(sp * 4);
  t += 2 * r(3 * sp * sp * 2) + r(3 * (size_t)c * sp * 2);
  t += r(64) + r(prepare_workspace_bytes((int64_t)sp));
  if (alpha > 0.0) t += r(outlier_extra_bytes(c, b));
  return t + 256;
}

thanos_status_t prune_layer_structured_impl(const void* W_in, void* W_out, uint8_t* col_removed_out,
                                            uint8_t* row_outlier_out, thanos_dtype_t wdtype,
                                            int64_t c, int64_t b, const float* U,
                                            const float* xnorm, const float* H, double p,
                                            double alpha, void* workspace, size_t ws_bytes,
                                            thanos_stats_t* stats, cudaStream_t stream) {
  const int64_t s = structured_column_count(p, b, alpha);
  if (s < 0 || s >= b) return THANOS_ERR_INVALID_ARG;
  const int64_t sp = padded(s);
  if (sp > b) return THANOS_ERR_SHAPE;
  const bool need_wc = wdtype != THANOS_F32;
  const bool need_outl = alpha > 0.0;
  const int n_out = need_outl ? (int)ceil(alpha * (double)c - 1e-12) : 0;
  StructWs w;
  if (!carve_struct(w, workspace, ws_bytes, c, b, sp, need_wc, need_outl))
    return THANOS_ERR_WORKSPACE;
  const int64_t nel = c * b;
  float* Wc;
  if (need_wc) {
    Wc = w.Wc;
    THANOS_TRY(convert_to_f32(static_cast<const __nv_bfloat16*>(W_in), Wc, nel, stream));
  } else {
    Wc = static_cast<float*>(W_out);
    if (W_in != W_out)
      THANOS_CUDA(cudaMemcpyAsync(W_out, W_in, (size_t)nel * sizeof(float),
                                  cudaMemcpyDeviceToDevice, stream));
  }
  THANOS_CUDA(cudaMemsetAsync(w.status, 0, 64, stream));
  int32_t* prep_status = w.status;
  int32_t* tc_status = w.status + 4;
  // ---- outlier rows
  const uint8_t* flags = w.flags;
  if (need_outl) {
    uint8_t* f = nullptr;
    THANOS_TRY(outlier_row_flags(Wc, H, c, b, n_out, w.outl, w.outl_bytes, &f, tc_status, stream));
    flags = f;
  } else {
    THANOS_CUDA(cudaMemsetAsync(w.flags, 0, (size_t)c, stream));
  }
  if (row_outlier_out)
    THANOS_CUDA(cudaMemcpyAsync(row_outlier_out, flags, (size_t)c, cudaMemcpyDeviceToDevice,
                                stream));
  // ---- the s columns of smallest loss
  const int chunks = (int)ceil_div(c, ROW_CHUNK);
  const unsigned bcols = (unsigned)ceil_div(b, 256);
  col_sq_partial_kernel<<<dim3((unsigned)chunks, bcols), 256, 0, stream>>>(Wc, flags, (int)c,
                                                                          (int)b, w.partial);
  THANOS_CHECK_LAUNCH();
  col_loss_kernel<<<bcols, 256, 0, stream>>>(w.partial, chunks, xnorm, (int)b, w.v);
  THANOS_CHECK_LAUNCH();
  smallest_cols_kernel<<<1, 1024, 0, stream>>>(w.v, (int)b, (int)s, (int)sp, w.colrm, w.qlist);
  THANOS_CHECK_LAUNCH();
  if (col_removed_out)
    THANOS_CUDA(cudaMemcpyAsync(col_removed_out, w.colrm, (size_t)b, cudaMemcpyDeviceToDevice,
                                stream));
  if (s > 0) {
    const int64_t pl_sb = sp * b, pl_ss = sp * sp;
    // ---- R = (U[:, q])^T U
    gather_uq_kernel<<<dim3((unsigned)ceil_div(b, 32), (unsigned)ceil_div(sp, 32)), 256, 0,
                       stream>>>(U, (int)b, w.qlist, (int)sp, w.UqT);
    THANOS_CHECK_LAUNCH();
    THANOS_TRY(split3_planes(U, b, b, b, w.Up, b, b * b, stream));
    {
      TcGemmArgs g;
      g.D = w.R;
      g.ldd = b;
      g.Dp = w.Rp;
      g.ldp = b;
      g.dp_plane = pl_sb;
      g.A = w.UqT;
      g.lda = b;
      g.a_plane = pl_sb;
      g.B = w.Up;
      g.ldb = b;
      g.b_plane = b * b;
      g.b_kmajor = 0;
      g.b_upper = 1;
      g.M = (int)sp;
      g.N = (int)b;
      g.K = (int)b;
      g.status = tc_status;
      THANOS_TRY(tc_gemm_split3(g, stream));
    }
    // ---- Rhat = R[:, q] and its inverse factor
    gather_rhat_kernel<<<dim3((unsigned)sp, (unsigned)ceil_div(sp, 256)), 256, 0, stream>>>(
        w.R, (int)b, w.qlist, (int)sp, w.Rhat);
    THANOS_CHECK_LAUNCH();
    THANOS_TRY(prepare_inverse_impl(w.Rhat, sp, 0.f, w.Ur, w.xdummy, w.prep, w.prep_bytes,
                                    prep_status, stream));
    THANOS_TRY(split3_planes(w.Ur, sp, sp, sp, w.Urp, sp, pl_ss, stream));
    transpose_split_kernel<<<dim3((unsigned)ceil_div(sp, 32), (unsigned)ceil_div(sp, 32)), 256, 0,
                             stream>>>(w.Ur, (int)sp, w.UrTp);
    THANOS_CHECK_LAUNCH();
    // ---- Y = Ur^T (Ur R)
    {
      TcGemmArgs g;
      g.Dp = w.Zp;
      g.ldp = b;
      g.dp_plane = pl_sb;
      g.A = w.Urp;
      g.lda = sp;
      g.a_plane = pl_ss;
      g.a_upper = 1;
      g.B = w.Rp;
      g.ldb = b;
      g.b_plane = pl_sb;
      g.b_kmajor = 0;
      g.M = (int)sp;
      g.N = (int)b;
      g.K = (int)sp;
      g.status = tc_status;
      THANOS_TRY(tc_gemm_split3(g, stream));
      g.Dp = w.Yp;
      g.A = w.UrTp;
      g.a_upper = 0;
      g.B = w.Zp;
      THANOS_TRY(tc_gemm_split3(g, stream));
    }
    // ---- W -= W[:, q] Y on the pruned rows, then exact zeros in the removed columns
    gather_wq_kernel<<<dim3((unsigned)c, (unsigned)ceil_div(sp, 256)), 256, 0, stream>>>(
        Wc, flags, (int)c, (int)b, w.qlist, (int)sp, w.Wqp);
    THANOS_CHECK_LAUNCH();
    {
      TcGemmArgs g;
      g.D = Wc;
      g.ldd = b;
      g.A = w.Wqp;
      g.lda = sp;
      g.a_plane = c * sp;
      g.B = w.Yp;
      g.ldb = b;
      g.b_plane = pl_sb;
      g.b_kmajor = 0;
      g.M = (int)c;
      g.N = (int)b;
      g.K = (int)sp;
      g.alpha = -1.f;
      g.accumulate = 1;
      g.status = tc_status;
      THANOS_TRY(tc_gemm_split3(g, stream));
    }
    zero_removed_kernel<<<dim3((unsigned)c, bcols), 256, 0, stream>>>(Wc, flags, w.colrm, (int)c,
                                                                      (int)b);
    THANOS_CHECK_LAUNCH();
  }
  finish_kernel<<<1, 1, 0, stream>>>(stats, prep_status, tc_status,
                                     (long long)s * (long long)(c - n_out), (int)s);
  THANOS_CHECK_LAUNCH();
  if (need_wc) {
    THANOS_TRY(convert_to_bf16(Wc, static_cast<__nv_bfloat16*>(W_out), nel, stream));
  }
  return THANOS_OK;
}

}  // namespace thanos
