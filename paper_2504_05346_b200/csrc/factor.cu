// thanos_prepare_inverse: one factorisation that yields the inverse of every trailing block of
// the damped Hessian (replaces the per-block re-inversion of Algorithm 1's last loop line).
//
//   H_d = H + lambda I = V V^T   with V upper-triangular (Cholesky taken from the LAST row /
//   column backwards), U = V^{-1} (upper).  Then H_d^{-1} = U^T U and, because V[j:, j:] is the
//   same kind of factor of H_d[j:, j:], inv(H_d[j:, j:]) = U[j:, j:]^T U[j:, j:] for every j.
//
// Blocked right-looking factorisation with NB-wide panels (diagonal blocks in float64 inside
// one CTA), then a divide-and-conquer triangular inverse whose levels are batched GEMMs.
#include "simt_gemm.cuh"

namespace thanos {

namespace {

constexpr int NB = 64;

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

// ---- diagonal block: V22 V22^T = A22 (upper, reversed order) and its inverse, in float64 ----
__global__ void __launch_bounds__(256)
potrf_diag_kernel(float* __restrict__ V, int b, int k0, int n, float* __restrict__ Dinv,
                  int32_t* __restrict__ status) {
  extern __shared__ __align__(16) unsigned char potrf_smem[];
  double (*S)[NB + 1] = reinterpret_cast<double (*)[NB + 1]>(potrf_smem);
  double (*Si)[NB + 1] = S + NB;
  const int tid = threadIdx.x;
  for (int e = tid; e < NB * NB; e += 256) {
    int i = e / NB, j = e % NB;
    double v = 0.0;
    if (i < n && j < n) {
      int a = i < j ? i : j, c = i < j ? j : i;
      v = (double)V[(int64_t)(k0 + a) * b + k0 + c];
    }
    S[i][j] = v;
    Si[i][j] = 0.0;
  }
  __syncthreads();
  for (int k = n - 1; k >= 0; --k) {
    double piv = S[k][k];
    bool bad = !(piv > 0.0) || !isfinite(piv);
    if (bad) {
      if (tid == 0) report_error(status, THANOS_ERR_NOT_SPD, k0 + k);
      piv = 1.0;
    }
    double d = sqrt(piv);
    __syncthreads();
    if (tid == 0) S[k][k] = d;
    for (int i = tid; i < k; i += 256) S[i][k] = S[i][k] / d;
    __syncthreads();
    // trailing (leading, in this order) update of the upper triangle i <= j < k
    for (int e = tid; e < k * k; e += 256) {
      int i = e / k, j = e % k;
      if (i <= j) S[i][j] -= S[i][k] * S[j][k];
    }
    __syncthreads();
  }
  // inverse of the upper-triangular block, one column per thread (back substitution)
  if (tid < n) {
    const int cidx = tid;
    for (int i = n - 1; i >= 0; --i) {
      double x;
      if (i > cidx) {
        x = 0.0;
      } else {
        double acc = (i == cidx) ? 1.0 : 0.0;
        for (int j = i + 1; j <= cidx; ++j) acc -= S[i][j] * Si[j][cidx];
        x = acc / S[i][i];
      }
      Si[i][cidx] = x;
    }
  }
  __syncthreads();
  for (int e = tid; e < NB * NB; e += 256) {
    int i = e / NB, j = e % NB;
    if (i < n && j < n) {
      if (j >= i) V[(int64_t)(k0 + i) * b + k0 + j] = (float)S[i][j];
      Dinv[i * NB + j] = (j >= i) ? (float)Si[i][j] : 0.f;
    } else {
      Dinv[i * NB + j] = 0.f;
    }
  }
}

// ---- panel: V12 = A12 * V22^{-T}, rows [0, k0), in place -----------------------------------
__global__ void __launch_bounds__(256)
trsm_panel_kernel(float* __restrict__ V, int b, int k0, int n, const float* __restrict__ Dinv) {
  using G = SimtGemm<64, 64, 16, 4, 4, false, true, float, float>;
  __shared__ float smem[G::SMEM_FLOATS];
  float acc[4][4] = {};
  int m0 = blockIdx.x * 64;
  // out(m, j) = sum_k A12(m, k) * Dinv(j, k)
  G::run(V + k0, b, Dinv, NB, k0, n, m0, 0, 0, n, acc, smem);
  const int tx = threadIdx.x % G::TX, ty = threadIdx.x / G::TX;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int gm = m0 + G::row_of(ty, i);
    if (gm >= k0) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int gn = G::col_of(tx, j);
      if (gn < n) V[(int64_t)gm * b + k0 + gn] = acc[i][j];
    }
  }
}

// ---- trailing update: A11 -= V12 V12^T on upper-triangle tiles ------------------------------
__global__ void __launch_bounds__(256)
syrk_trailing_kernel(float* __restrict__ V, int b, int k0, int n, int nt) {
  using G = SimtGemm<128, 128, 16, 8, 8, false, true, float, float>;
  __shared__ float smem[G::SMEM_FLOATS];
  int p = blockIdx.x, I = 0;
  while (p >= nt - I) {
    p -= nt - I;
    ++I;
  }
  int J = I + p;
  float acc[8][8];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;
  G::run(V + k0, b, V + k0, b, k0, k0, I * 128, J * 128, 0, n, acc, smem);
  const int tx = threadIdx.x % G::TX, ty = threadIdx.x / G::TX;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    int gm = I * 128 + G::row_of(ty, i);
    if (gm >= k0) continue;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      int gn = J * 128 + G::col_of(tx, j);
      if (gn < k0 && gn >= gm) V[(int64_t)gm * b + gn] -= acc[i][j];
    }
  }
}

// ---- U initialisation: inverted diagonal blocks, zero elsewhere -----------------------------
__global__ void init_inverse_kernel(float* __restrict__ U, int b, const float* __restrict__ Dinv) {
  int j = blockIdx.x * blockDim.x + threadIdx.x;
  int i = blockIdx.y;
  if (j >= b) return;
  float v = 0.f;
  if (i / NB == j / NB) v = Dinv[(int64_t)(i / NB) * NB * NB + (i % NB) * NB + (j % NB)];
  U[(int64_t)i * b + j] = v;
}

// Level of the divide-and-conquer inverse: for pair t with halves [r0, c0) and [c0, c0 + N):
//   T = V12 * U22   (U22 upper: k <= n)        then        U12 = -U11 * T   (U11 upper: k >= m)
template <int BT, int TT>
__global__ void __launch_bounds__((BT / TT) * (BT / TT))
trinv_gemm1_kernel(const float* __restrict__ V, const float* __restrict__ U,
                   float* __restrict__ T, int b, int sz) {
  using G = SimtGemm<BT, BT, 16, TT, TT, false, false, float, float>;
  __shared__ float smem[G::SMEM_FLOATS];
  int t = blockIdx.z;
  int64_t r0 = (int64_t)2 * t * sz, c0 = r0 + sz;
  if (c0 >= b) return;
  int N = (int)((c0 + sz < b ? c0 + sz : b) - c0);
  int m0 = blockIdx.y * BT, n0 = blockIdx.x * BT;
  if (m0 >= sz || n0 >= N) return;
  float acc[TT][TT];
#pragma unroll
  for (int i = 0; i < TT; ++i)
#pragma unroll
    for (int j = 0; j < TT; ++j) acc[i][j] = 0.f;
  int kend = n0 + BT < N ? n0 + BT : N;
  G::run(V + r0 * b + c0, b, U + c0 * b + c0, b, sz, N, m0, n0, 0, kend, acc, smem);
  float* Tt = T + (int64_t)t * sz * sz;  // every pair before the last has N == sz
  const int tx = threadIdx.x % G::TX, ty = threadIdx.x / G::TX;
#pragma unroll
  for (int i = 0; i < TT; ++i) {
    int gm = m0 + G::row_of(ty, i);
    if (gm >= sz) continue;
#pragma unroll
    for (int j = 0; j < TT; ++j) {
      int gn = n0 + G::col_of(tx, j);
      if (gn < N) Tt[(int64_t)gm * N + gn] = acc[i][j];
    }
  }
}

template <int BT, int TT>
__global__ void __launch_bounds__((BT / TT) * (BT / TT))
trinv_gemm2_kernel(float* __restrict__ U, const float* __restrict__ T, int b, int sz) {
  using G = SimtGemm<BT, BT, 16, TT, TT, false, false, float, float>;
  __shared__ float smem[G::SMEM_FLOATS];
  int t = blockIdx.z;
  int64_t r0 = (int64_t)2 * t * sz, c0 = r0 + sz;
  if (c0 >= b) return;
  int N = (int)((c0 + sz < b ? c0 + sz : b) - c0);
  int m0 = blockIdx.y * BT, n0 = blockIdx.x * BT;
  if (m0 >= sz || n0 >= N) return;
  float acc[TT][TT];
#pragma unroll
  for (int i = 0; i < TT; ++i)
#pragma unroll
    for (int j = 0; j < TT; ++j) acc[i][j] = 0.f;
  const float* Tt = T + (int64_t)t * sz * sz;
  G::run(U + r0 * b + r0, b, Tt, N, sz, N, m0, n0, m0, sz, acc, smem);
  const int tx = threadIdx.x % G::TX, ty = threadIdx.x / G::TX;
#pragma unroll
  for (int i = 0; i < TT; ++i) {
    int gm = m0 + G::row_of(ty, i);
    if (gm >= sz) continue;
#pragma unroll
    for (int j = 0; j < TT; ++j) {
      int gn = n0 + G::col_of(tx, j);
      if (gn < N) U[(r0 + gm) * b + c0 + gn] = -acc[i][j];
    }
  }
}

}  // namespace

size_t prepare_workspace_bytes(int64_t b) {
  size_t nblk = (size_t)ceil_div(b, NB);
  size_t v = round_up((size_t)b * b * sizeof(float), 256);
  size_t d = round_up(nblk * NB * NB * sizeof(float), 256);
  size_t t = round_up(((size_t)b * b / 4 + (size_t)b * NB) * sizeof(float), 256);
  return v + d + t + 256;
}

thanos_status_t prepare_inverse_impl(const float* H, int64_t b64, float damp_rel, float* factor,
                                     float* xnorm, void* workspace, size_t ws_bytes,
                                     int32_t* status_dev, cudaStream_t stream) {
  const int b = (int)b64;
  Arena ar(workspace, ws_bytes);
  int nblk = (int)ceil_div(b, NB);
  float* V = ar.take<float>((size_t)b * b);
  float* Dinv = ar.take<float>((size_t)nblk * NB * NB);
  float* T = ar.take<float>((size_t)b * b / 4 + (size_t)b * NB);
  float* lam = ar.take<float>(1);
  if (!ar.ok()) return THANOS_ERR_WORKSPACE;

  diag_stats_kernel<<<1, 1024, 0, stream>>>(H, b, damp_rel, xnorm, lam);
  THANOS_CHECK_LAUNCH();
  dim3 cg((unsigned)ceil_div(b, 256), (unsigned)b);
  copy_damped_upper_kernel<<<cg, 256, 0, stream>>>(H, V, b, lam);
  THANOS_CHECK_LAUNCH();

  constexpr int POTRF_SMEM = 2 * NB * (NB + 1) * (int)sizeof(double);
  THANOS_CUDA(cudaFuncSetAttribute(potrf_diag_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   POTRF_SMEM));
  for (int kb = nblk - 1; kb >= 0; --kb) {
    int k0 = kb * NB;
    int n = (b - k0 < NB) ? b - k0 : NB;
    float* Dk = Dinv + (size_t)kb * NB * NB;
    potrf_diag_kernel<<<1, 256, POTRF_SMEM, stream>>>(V, b, k0, n, Dk, status_dev);
    THANOS_CHECK_LAUNCH();
    if (k0 > 0) {
      trsm_panel_kernel<<<(unsigned)ceil_div(k0, 64), 256, 0, stream>>>(V, b, k0, n, Dk);
      THANOS_CHECK_LAUNCH();
      int nt = (int)ceil_div(k0, 128);
      syrk_trailing_kernel<<<nt * (nt + 1) / 2, 256, 0, stream>>>(V, b, k0, n, nt);
      THANOS_CHECK_LAUNCH();
    }
  }

  init_inverse_kernel<<<cg, 256, 0, stream>>>(factor, b, Dinv);
  THANOS_CHECK_LAUNCH();
  for (int64_t sz = NB; sz < b; sz *= 2) {
    int npairs = (int)ceil_div(b, 2 * sz);
    if (sz <= 64) {
      dim3 g((unsigned)ceil_div(sz, 64), (unsigned)ceil_div(sz, 64), (unsigned)npairs);
      trinv_gemm1_kernel<64, 4><<<g, 256, 0, stream>>>(V, factor, T, b, (int)sz);
      THANOS_CHECK_LAUNCH();
      trinv_gemm2_kernel<64, 4><<<g, 256, 0, stream>>>(factor, T, b, (int)sz);
      THANOS_CHECK_LAUNCH();
    } else {
      dim3 g((unsigned)ceil_div(sz, 128), (unsigned)ceil_div(sz, 128), (unsigned)npairs);
      trinv_gemm1_kernel<128, 8><<<g, 256, 0, stream>>>(V, factor, T, b, (int)sz);
      THANOS_CHECK_LAUNCH();
      trinv_gemm2_kernel<128, 8><<<g, 256, 0, stream>>>(factor, T, b, (int)sz);
      THANOS_CHECK_LAUNCH();
    }
  }
  return THANOS_OK;
}

}  // namespace thanos
