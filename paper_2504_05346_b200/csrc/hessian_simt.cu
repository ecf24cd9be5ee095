// H += 2 X^T X on the plain fp32 ALUs (Section 3.2: H = 2 X X^T with the paper's X = our X^T).
// Generic path: any dtype, any shape, exact fp32 products.  Upper-triangle tiles only; the
// mirror tile is written from the same accumulators.
#include "simt_gemm.cuh"

namespace thanos {

namespace {

constexpr int HB = 128;  // tile edge
constexpr int HK = 16;

template <typename T>
__global__ void __launch_bounds__(256)
hessian_syrk_simt_kernel(float* __restrict__ H, int b, const T* __restrict__ X, int64_t ldx,
                         int64_t n_tok, int nt, int64_t tok_per_slice) {
  using G = SimtGemm<HB, HB, HK, 8, 8, true, false, T, T>;
  __shared__ float smem[G::SMEM_FLOATS];
  // upper-triangle tile pair (I <= J) from the linear index
  int p = blockIdx.x;
  int I = 0;
  while (p >= nt - I) {
    p -= nt - I;
    ++I;
  }
  int J = I + p;
  int64_t t0 = (int64_t)blockIdx.y * tok_per_slice;
  int64_t t1 = t0 + tok_per_slice;
  if (t1 > n_tok) t1 = n_tok;
  if (t0 >= t1) return;
  float acc[8][8];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;
  // A(m, k) = X[k, I*HB + m] (transposed read), B(k, n) = X[k, J*HB + n]
  const T* Xs = X + t0 * ldx;
  G::run(Xs, ldx, Xs, ldx, b, b, I * HB, J * HB, 0, (int)(t1 - t0), acc, smem);
  const int tx = threadIdx.x % G::TX, ty = threadIdx.x / G::TX;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    int gi = I * HB + G::row_of(ty, i);
    if (gi >= b) continue;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      int gj = J * HB + G::col_of(tx, j);
      if (gj >= b) continue;
      float v = 2.f * acc[i][j];
      atomicAdd(&H[(int64_t)gi * b + gj], v);
      if (I != J) atomicAdd(&H[(int64_t)gj * b + gi], v);
    }
  }
}

}  // namespace

thanos_status_t hessian_accumulate_simt(float* H, int64_t b, const void* X, thanos_dtype_t xdtype,
                                        int64_t n_tok, int64_t ldx, cudaStream_t stream,
                                        bool ordered) {
  int nt = (int)ceil_div(b, HB);
  int npairs = nt * (nt + 1) / 2;
  // slice tokens so the grid has a few waves of CTAs; each slice is at most 2^30 tokens
  // ordered: one slice, so that every entry of H receives exactly one addend per call
  int64_t want_slices = ordered ? 1 : ceil_div(NUM_SMS * 4, npairs);
  int64_t tok_per_slice = ceil_div(n_tok, want_slices);
  tok_per_slice = round_up((size_t)(tok_per_slice < 256 ? 256 : tok_per_slice), HK);
  if (tok_per_slice > (1 << 30)) tok_per_slice = 1 << 30;
  int64_t slices = ceil_div(n_tok, tok_per_slice);
  if (ordered && slices != 1) return THANOS_ERR_SHAPE;
  if (slices > 65535) return THANOS_ERR_SHAPE;
  dim3 grid(npairs, (unsigned)slices);
  if (xdtype == THANOS_F32) {
    hessian_syrk_simt_kernel<float><<<grid, 256, 0, stream>>>(
        H, (int)b, static_cast<const float*>(X), ldx, n_tok, nt, tok_per_slice);
  } else {
    hessian_syrk_simt_kernel<__nv_bfloat16><<<grid, 256, 0, stream>>>(
        H, (int)b, static_cast<const __nv_bfloat16*>(X), ldx, n_tok, nt, tok_per_slice);
  }
  THANOS_CHECK_LAUNCH();
  return THANOS_OK;
}

}  // namespace thanos
