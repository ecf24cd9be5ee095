// thanos_prepare_inverse: one factorisation that yields the inverse of every trailing block of
// the damped Hessian (replaces the per-block re-inversion of Algorithm 1's last loop line).
//
//   H_d = H + lambda I = V V^T   with V upper-triangular (Cholesky taken from the LAST row /
//   column backwards), U = V^{-1} (upper).  Then H_d^{-1} = U^T U and, because V[j:, j:] is the
//   same kind of factor of H_d[j:, j:], inv(H_d[j:, j:]) = U[j:, j:]^T U[j:, j:] for every j.
//
// Blocked right-looking factorisation with 128-wide panels: the 128 x 128 diagonal block is
// factored and inverted by one CTA, the panel and the trailing update are tensor-core products
// (three bf16 planes per operand, see tc_gemm.cuh); then a divide-and-conquer triangular inverse
// whose levels are tensor-core products as well.
#include "simt_gemm.cuh"
#include "tc_gemm.cuh"

namespace thanos {

namespace {

constexpr int NB = 128;
constexpr int DLD = NB + 4;  // row stride of the diagonal-block scratch (odd multiple of 16 bytes)

// ---- mean(diag H) -> lambda, xnorm ---------------------------------------------------------
__global__ void __launch_bounds__(1024)
diag_stats_kernel(const float* __restrict__ H, int b, float damp_rel, float* __restrict__ xnorm,
                  float* __restrict__ lam_out) {
  __shared__ double red[32];
  double s = 0.0;
  for (int j = threadIdx.x; j < b; j += blockDim.x) {
    float d = H[(int64_t)j * b + j];
    xnorm[j] = sqrtf(fmaxf(d, 0.f) * 0.5f);
    s += (double)d;
  }
  for (int o = 16; o > 0; o >>= 1) s += __shfl_down_sync(0xffffffffu, s, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = s;
  __syncthreads();
  if (threadIdx.x < 32) {
    double t = (threadIdx.x < (blockDim.x >> 5)) ? red[threadIdx.x] : 0.0;
    for (int o = 16; o > 0; o >>= 1) t += __shfl_down_sync(0xffffffffu, t, o);
    if (threadIdx.x == 0) *lam_out = (float)((double)damp_rel * (t / (double)b));
  }
}

// V <- upper triangle of H (+ lambda on the diagonal); below the diagonal 0.
__global__ void copy_damped_upper_kernel(const float* __restrict__ H, float* __restrict__ V, int b,
                                         const float* __restrict__ lam) {
  int j = blockIdx.x * blockDim.x + threadIdx.x;
  int i = blockIdx.y;
  if (j >= b) return;
  float v = 0.f;
  if (j >= i) {
    v = H[(int64_t)i * b + j];
    if (i == j) v += *lam;
  }
  V[(int64_t)i * b + j] = v;
}

// ---- diagonal block: A22 = V22 V22^T (V22 upper, i.e. Cholesky from the last row backwards) and
//      U22 = inv(V22).  One CTA.  With the rows and columns reversed this is an ordinary lower
//      Cholesky L; n identity rows appended below the block turn into L^{-T} under the same
//      elimination, which gives the inverse without a second pass.
//      Left-looking in panels of 8 columns.  Two threads share a row and split the contraction
//      range in alternating runs of 16 columns; every thread factors the 8 x 8 diagonal piece
//      itself (reciprocal square roots by one Newton step on the hardware estimate).
constexpr int DIAG_THREADS = 4 * NB;

__global__ void __launch_bounds__(DIAG_THREADS)
diag_block_kernel(float* __restrict__ V, float* __restrict__ U, __nv_bfloat16* __restrict__ Up,
                  int64_t plane, int b, int k0, int n, int32_t* __restrict__ status) {
  extern __shared__ __align__(16) float dsm[];
  float* L = dsm;                       // [2 n][DLD]
  float* dblk = dsm + 2 * NB * DLD;     // [8][8]
  const int tid = threadIdx.x;
  const int warp = tid >> 5, lane = tid & 31;
  // reversed lower triangle of the block, then the identity
  for (int i = warp; i < n; i += DIAG_THREADS / 32) {
    const float* src = V + (int64_t)(k0 + n - 1 - i) * b + k0;
    for (int c4 = lane * 4; c4 < n; c4 += 128) {
      const float4 v = *reinterpret_cast<const float4*>(src + c4);
      const float e[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int j = n - 1 - (c4 + u);
        L[i * DLD + j] = (j <= i) ? e[u] : 0.f;
        L[(n + i) * DLD + j] = (i == j) ? 1.f : 0.f;
      }
    }
  }
  __syncthreads();
  const int r = tid >> 1;
  const int half = tid & 1;
  const bool is_row = r < 2 * n;
  float* Lr = L + (is_row ? r : 0) * DLD;
  // identity row j is zero left of column j: its products start there (rounded down to 32)
  const int first_nz = (r >= n) ? ((r - n) & ~31) : 0;
  for (int c0 = 0; c0 < n; c0 += 8) {
    const bool active = is_row && r >= c0;
    float acc[8];
    if (half == 0) {
      const float4 lo = *reinterpret_cast<const float4*>(Lr + c0);
      const float4 hi = *reinterpret_cast<const float4*>(Lr + c0 + 4);
      acc[0] = lo.x; acc[1] = lo.y; acc[2] = lo.z; acc[3] = lo.w;
      acc[4] = hi.x; acc[5] = hi.y; acc[6] = hi.z; acc[7] = hi.w;
    } else {
#pragma unroll
      for (int w = 0; w < 8; ++w) acc[w] = 0.f;
    }
    if (active) {
      const float* Pb = L + c0 * DLD;
      for (int kk = first_nz + 16 * half; kk < c0; kk += 32) {
        const int kend = kk + 16 < c0 ? kk + 16 : c0;
        for (int k = kk; k < kend; k += 4) {
          const float4 av = *reinterpret_cast<const float4*>(Lr + k);
#pragma unroll
          for (int w = 0; w < 8; ++w) {
            const float4 bv = *reinterpret_cast<const float4*>(Pb + w * DLD + k);
            acc[w] = fmaf(-av.x, bv.x, acc[w]);
            acc[w] = fmaf(-av.y, bv.y, acc[w]);
            acc[w] = fmaf(-av.z, bv.z, acc[w]);
            acc[w] = fmaf(-av.w, bv.w, acc[w]);
          }
        }
      }
    }
#pragma unroll
    for (int w = 0; w < 8; ++w) acc[w] += __shfl_xor_sync(0xffffffffu, acc[w], 1);
    if (half == 0 && r >= c0 && r < c0 + 8) {
#pragma unroll
      for (int w = 0; w < 8; ++w) dblk[(r - c0) * 8 + w] = acc[w];
    }
    __syncthreads();
    // 8 x 8 Cholesky of the diagonal piece, in registers, by every thread
    float ld[8][8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
      for (int j = 0; j <= i; ++j) ld[i][j] = dblk[i * 8 + j];
    float rinv[8];
#pragma unroll
    for (int w = 0; w < 8; ++w) {
      float d = ld[w][w];
      if (!(d > 0.f) || !isfinite(d)) {
        if (tid == 0) report_error(status, THANOS_ERR_NOT_SPD, k0 + n - 1 - (c0 + w));
        d = 1.f;
      }
      float ri = rsqrtf(d);
      ri = ri * fmaf(-0.5f * d, ri * ri, 1.5f);
      rinv[w] = ri;
#pragma unroll
      for (int v = w; v < 8; ++v) ld[v][w] *= ri;
#pragma unroll
      for (int v = w + 1; v < 8; ++v)
#pragma unroll
        for (int u = w + 1; u <= v; ++u) ld[v][u] = fmaf(-ld[v][w], ld[u][w], ld[v][u]);
    }
    // this thread's row: x L_d^T = acc
    float x[8];
#pragma unroll
    for (int w = 0; w < 8; ++w) {
      float t = acc[w];
#pragma unroll
      for (int v = 0; v < w; ++v) t = fmaf(-x[v], ld[w][v], t);
      x[w] = t * rinv[w];
    }
    if (active && half == 0) {
      *reinterpret_cast<float4*>(Lr + c0) = make_float4(x[0], x[1], x[2], x[3]);
      *reinterpret_cast<float4*>(Lr + c0 + 4) = make_float4(x[4], x[5], x[6], x[7]);
    }
    __syncthreads();
  }
  // V22[i][j] = L[n-1-i][n-1-j];  U22[i][j] = inv(L)[n-1-i][n-1-j] = extra row (n-1-j), column n-1-i
  for (int i = warp; i < n; i += DIAG_THREADS / 32) {
    for (int c4 = lane * 4; c4 < n; c4 += 128) {
      float u4[4];
      const int64_t o = (int64_t)(k0 + i) * b + k0 + c4;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int j = c4 + e;
        float u = 0.f;
        if (j >= i) {
          V[o + e] = L[(n - 1 - i) * DLD + (n - 1 - j)];
          u = L[(n + n - 1 - j) * DLD + (n - 1 - i)];
        }
        u4[e] = u;
      }
      *reinterpret_cast<float4*>(U + o) = make_float4(u4[0], u4[1], u4[2], u4[3]);
#pragma unroll
      for (int pl = 0; pl < 3; ++pl) {
        __nv_bfloat16 hb[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          hb[e] = __float2bfloat16_rn(u4[e]);
          u4[e] -= __bfloat162float(hb[e]);
        }
        uint2 pk;
        pk.x = (uint32_t)__bfloat16_as_ushort(hb[0]) | ((uint32_t)__bfloat16_as_ushort(hb[1]) << 16);
        pk.y = (uint32_t)__bfloat16_as_ushort(hb[2]) | ((uint32_t)__bfloat16_as_ushort(hb[3]) << 16);
        *reinterpret_cast<uint2*>(Up + (int64_t)pl * plane + o) = pk;
      }
    }
  }
}

__global__ void fold_status_kernel(const int32_t* tc_status, int32_t* status) {
  if (*tc_status != 0) atomicCAS(status, 0, *tc_status);
}

struct PrepareWs {
  float* V;
  __nv_bfloat16* Vp;
  __nv_bfloat16* Up;
  __nv_bfloat16* Tp;
  size_t t_elems;
  float* lam;
  int32_t* tc_status;
};

size_t t_plane_elems(int64_t b) { return (size_t)b * b / 4 + (size_t)b * NB + 64; }

bool carve_prepare(PrepareWs& w, void* workspace, size_t ws_bytes, int64_t b) {
  Arena ar(workspace, ws_bytes);
  w.V = ar.take<float>((size_t)b * b);
  w.Vp = ar.take<__nv_bfloat16>(3 * (size_t)b * b);
  w.Up = ar.take<__nv_bfloat16>(3 * (size_t)b * b);
  w.t_elems = round_up(t_plane_elems(b), 64);
  w.Tp = ar.take<__nv_bfloat16>(3 * w.t_elems);
  w.lam = ar.take<float>(1);
  w.tc_status = ar.take<int32_t>(4);
  return ar.ok();
}

}  // namespace

size_t prepare_workspace_bytes(int64_t b) {
  size_t t = round_up((size_t)b * b * sizeof(float), 256);
  t += 2 * round_up(3 * (size_t)b * b * sizeof(__nv_bfloat16), 256);
  t += round_up(3 * round_up(t_plane_elems(b), 64) * sizeof(__nv_bfloat16), 256);
  return t + 3 * 256;
}

thanos_status_t prepare_inverse_impl(const float* H, int64_t b64, float damp_rel, float* factor,
                                     float* xnorm, void* workspace, size_t ws_bytes,
                                     int32_t* status_dev, cudaStream_t stream) {
  const int b = (int)b64;
  PrepareWs w;
  if (!carve_prepare(w, workspace, ws_bytes, b)) return THANOS_ERR_WORKSPACE;
  const int64_t plane = (int64_t)b * b;
  const int nblk = (int)ceil_div(b, NB);

  diag_stats_kernel<<<1, 1024, 0, stream>>>(H, b, damp_rel, xnorm, w.lam);
  THANOS_CHECK_LAUNCH();
  dim3 cg((unsigned)ceil_div(b, 256), (unsigned)b);
  copy_damped_upper_kernel<<<cg, 256, 0, stream>>>(H, w.V, b, w.lam);
  THANOS_CHECK_LAUNCH();
  THANOS_CUDA(cudaMemsetAsync(factor, 0, (size_t)plane * sizeof(float), stream));
  THANOS_CUDA(cudaMemsetAsync(w.Up, 0, 3 * (size_t)plane * sizeof(__nv_bfloat16), stream));
  THANOS_CUDA(cudaMemsetAsync(w.tc_status, 0, 16, stream));

  constexpr int DIAG_SMEM = (2 * NB * DLD + 64) * (int)sizeof(float);
  {
    static std::atomic<unsigned long long> done{0};
    THANOS_CUDA(ensure_max_dyn_smem(diag_block_kernel, DIAG_SMEM, done));
  }
  // ---- H_d = V V^T, panels from the last one backwards
  for (int kb = nblk - 1; kb >= 0; --kb) {
    const int k0 = kb * NB;
    const int n = (b - k0 < NB) ? b - k0 : NB;
    diag_block_kernel<<<1, DIAG_THREADS, DIAG_SMEM, stream>>>(w.V, factor, w.Up, plane, b, k0, n,
                                                       status_dev);
    THANOS_CHECK_LAUNCH();
    if (k0 == 0) break;
    // V12 = A12 U22^T (rows above the block), written over A12 and as planes
    THANOS_TRY(split3_planes(w.V + k0, b, k0, n, w.Vp + k0, b, plane, stream));
    TcGemmArgs g;
    g.D = w.V + k0;
    g.ldd = b;
    g.Dp = w.Vp + k0;
    g.ldp = b;
    g.dp_plane = plane;
    g.A = w.Vp + k0;
    g.lda = b;
    g.a_plane = plane;
    g.B = w.Up + (int64_t)k0 * b + k0;
    g.ldb = b;
    g.b_plane = plane;
    g.b_kmajor = 1;
    g.M = k0;
    g.N = n;
    g.K = n;
    g.status = w.tc_status;
    THANOS_TRY(tc_gemm_split3(g, stream));
    // A11 -= V12 V12^T on the tiles that touch the upper triangle
    TcGemmArgs y;
    y.D = w.V;
    y.ldd = b;
    y.A = w.Vp + k0;
    y.lda = b;
    y.a_plane = plane;
    y.B = w.Vp + k0;
    y.ldb = b;
    y.b_plane = plane;
    y.b_kmajor = 1;
    y.M = k0;
    y.N = k0;
    y.K = n;
    y.alpha = -1.f;
    y.accumulate = 1;
    y.upper_only = 1;
    y.status = w.tc_status;
    THANOS_TRY(tc_gemm_split3(y, stream));
  }

  // ---- U = inv(V) by halves: for the pair of diagonal blocks [r0, c0) and [c0, c0 + N),
  //      U12 = -U11 (V12 U22)
  for (int64_t sz = NB; sz < b; sz *= 2) {
    const int npairs = (int)ceil_div(b, 2 * sz);
    // pairs whose second block is a full sz wide go out as one batched product per step; a
    // ragged last pair follows on its own
    int nfull = 0;
    while (nfull < npairs && (int64_t)(2 * nfull + 2) * sz <= b) ++nfull;
    for (int part = 0; part < 2; ++part) {
      const int t = part == 0 ? 0 : nfull;
      const int cnt = part == 0 ? nfull : npairs - nfull;
      if (cnt <= 0) continue;
      const int64_t r0 = 2 * t * sz, c0 = r0 + sz;
      if (c0 >= b) continue;
      const int N = (int)((c0 + sz < b ? c0 + sz : b) - c0);
      const int64_t pair_stride = 2 * sz * ((int64_t)b + 1);
      __nv_bfloat16* Tt = w.Tp + (size_t)t * sz * sz;
      TcGemmArgs g;
      g.Dp = Tt;
      g.ldp = N;
      g.dp_plane = (int64_t)w.t_elems;
      g.dp_batch = sz * sz;
      g.A = w.Vp + r0 * b + c0;
      g.lda = b;
      g.a_plane = plane;
      g.a_batch = pair_stride;
      g.B = w.Up + c0 * b + c0;
      g.ldb = b;
      g.b_plane = plane;
      g.b_batch = pair_stride;
      g.b_kmajor = 0;
      g.M = (int)sz;
      g.N = N;
      g.K = N;
      g.batch = part == 0 ? cnt : 1;
      g.b_upper = 1;  // U22 is upper-triangular
      g.status = w.tc_status;
      THANOS_TRY(tc_gemm_split3(g, stream));
      TcGemmArgs h;
      h.D = factor + r0 * b + c0;
      h.ldd = b;
      h.d_batch = pair_stride;
      h.Dp = w.Up + r0 * b + c0;
      h.ldp = b;
      h.dp_plane = plane;
      h.dp_batch = pair_stride;
      h.A = w.Up + r0 * b + r0;
      h.lda = b;
      h.a_plane = plane;
      h.a_batch = pair_stride;
      h.B = Tt;
      h.ldb = N;
      h.b_plane = (int64_t)w.t_elems;
      h.b_batch = sz * sz;
      h.b_kmajor = 0;
      h.M = (int)sz;
      h.N = N;
      h.K = (int)sz;
      h.batch = part == 0 ? cnt : 1;
      h.a_upper = 1;  // U11 is upper-triangular
      h.alpha = -1.f;
      h.status = w.tc_status;
      THANOS_TRY(tc_gemm_split3(h, stream));
    }
  }
  fold_status_kernel<<<1, 1, 0, stream>>>(w.tc_status, status_dev);
  THANOS_CHECK_LAUNCH();
  return THANOS_OK;
}

}  // namespace thanos
