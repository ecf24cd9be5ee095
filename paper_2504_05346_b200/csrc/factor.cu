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
#include "tile_ops.cuh"

namespace thanos {

namespace {

constexpr int NB = 128;
constexpr int PANEL_GROUP = 4;  // panels whose trailing updates go out as one product

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

// V <- upper triangle of H (+ lambda on the diagonal); below the diagonal 0.  Four columns per
// thread (b is a multiple of 8, so every row starts on a 16-byte boundary).
__global__ void copy_damped_upper_kernel(const float* __restrict__ H, float* __restrict__ V, int b,
                                         const float* __restrict__ lam) {
  const int j = 4 * (blockIdx.x * blockDim.x + threadIdx.x);
  const int i = blockIdx.y;
  if (j >= b) return;
  float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
  if (j + 3 >= i) {
    v = *reinterpret_cast<const float4*>(H + (int64_t)i * b + j);
    const float l = *lam;
    if (j < i) v.x = 0.f;
    if (j + 1 < i) v.y = 0.f;
    if (j + 2 < i) v.z = 0.f;
    if (j == i) v.x += l;
    if (j + 1 == i) v.y += l;
    if (j + 2 == i) v.z += l;
    if (j + 3 == i) v.w += l;
  }
  *reinterpret_cast<float4*>(V + (int64_t)i * b + j) = v;
}

// ---- diagonal block: A22 = V22 V22^T (V22 upper, i.e. Cholesky from the last row backwards) and
//      U22 = inv(V22).  One CTA.  With the rows and columns reversed this is an ordinary lower
//      Cholesky L; n identity rows appended below the block turn into L^{-T} under the same
//      elimination, which gives the inverse without a second pass.
//      The stacked matrix [reversed block; identity] lives in shared memory as 16 x 16 tiles
//      (2 Tn tile rows, Tn tile columns).  Right-looking: per tile column K the rows of the panel
//      are solved one thread per row, the trailing tiles are updated one warp per tile from a
//      shared counter, and warp 0 first brings the next diagonal tile up to date and factors it
//      (reciprocal square roots by one Newton step on the hardware estimate).  Identity row j
//      is zero left of column j, so its tiles join in from tile column j / 16 on.
constexpr int DIAG_THREADS = 512;
constexpr int DIAG_TILES = NB / 16;
constexpr int DIAG_SMEM = (2 * DIAG_TILES * DIAG_TILES * 256 + NB + 16) * (int)sizeof(float);

__global__ void __launch_bounds__(DIAG_THREADS, 1)
diag_block_kernel(float* __restrict__ V, float* __restrict__ U, __nv_bfloat16* __restrict__ Up,
                  int64_t plane, int b, int k0, int n, int32_t* __restrict__ status) {
  extern __shared__ __align__(16) float dsm[];
  const int Tn = (n + 15) >> 4;
  float* A = dsm;                                   // tile (I, J) at (I Tn + J) * 256
  float* invd = dsm + 2 * DIAG_TILES * DIAG_TILES * 256;  // [NB]
  unsigned* s_counter = reinterpret_cast<unsigned*>(invd + NB);
  const int tid = threadIdx.x;
  const int warp = tid >> 5, lane = tid & 31;
  auto tile_at = [&](int I, int J) { return A + ((I * Tn + J) << 8); };
  // zeros, with ones on the diagonal of the padding and of the identity rows ...
  for (int q = tid; q < 2 * Tn * Tn * 64; q += DIAG_THREADS) {
    const int t = q >> 6, r = (q >> 2) & 15, c = q & 3;
    const int I = t / Tn, J = t - I * Tn;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    const int d = r - 4 * c;  // the chunk holds the tile's diagonal element of row r at position d
    const bool diag_tile = I >= Tn ? (I - Tn == J) : (I == J && 16 * I + r >= n);
    if (diag_tile && d >= 0 && d < 4) {
      if (d == 0) v.x = 1.f;
      if (d == 1) v.y = 1.f;
      if (d == 2) v.z = 1.f;
      if (d == 3) v.w = 1.f;
    }
    *reinterpret_cast<float4*>(A + (t << 8) + tile::chunk_off(r, c)) = v;
  }
  __syncthreads();
  // ... then the reversed lower triangle of the block: a warp takes rows i, i + 16, ..., all of
  // its loads first
  {
    float4 v[NB / (DIAG_THREADS / 32)];
    const int c4 = lane * 4;
#pragma unroll
    for (int u = 0; u < NB / (DIAG_THREADS / 32); ++u) {
      const int i = warp + u * (DIAG_THREADS / 32);
      v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (i < n && c4 < n)
        v[u] = *reinterpret_cast<const float4*>(V + (int64_t)(k0 + n - 1 - i) * b + k0 + c4);
    }
#pragma unroll
    for (int u = 0; u < NB / (DIAG_THREADS / 32); ++u) {
      const int i = warp + u * (DIAG_THREADS / 32);
      if (i < n && c4 < n) {
        const float e4[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
        for (int w = 0; w < 4; ++w) {
          const int j = n - 1 - (c4 + w);
          if (j <= i) tile_at(i >> 4, j >> 4)[tile::elem_off(i & 15, j & 15)] = e4[w];
        }
      }
    }
  }
  __syncthreads();
  int bad = -1;
  if (warp == 0) bad = tile::factor_diag_tile<true>(tile_at(0, 0), invd, 0, n, lane);
  __syncthreads();
  for (int K = 0; K < Tn; ++K) {
    const int m = Tn - K - 1;  // tile rows of the block below the diagonal tile
    if (tid == 0) *s_counter = 1;
    // panel: the block's rows below the diagonal tile and the identity rows 0 .. 16 K + 15
    {
      const float* Lk = tile_at(K, K);
      for (int ii = tid; ii < 16 * (m + K + 1); ii += DIAG_THREADS) {
        const int tr = ii >> 4, r = ii & 15;
        const int I = tr < m ? K + 1 + tr : Tn + (tr - m);
        tile::panel_row_solve(tile_at(I, K), r, Lk, invd + 16 * K);
      }
    }
    __syncthreads();
    if (warp == 0 && K + 1 < Tn) {
      float* Ct = tile_at(K + 1, K + 1);
      tile::tile_update(Ct, tile_at(K + 1, K), tile_at(K + 1, K), lane);
      __syncwarp();
      const int bd = tile::factor_diag_tile<true>(Ct, invd, 16 * (K + 1), n, lane);
      if (bad < 0) bad = bd;
    }
    {
      // targets: the m (m + 1) / 2 tiles (I, J), K < J <= I, of the block (index 0 is the next
      // diagonal tile, done above), then the (K + 1) m tiles of the identity rows
      const int ntop = (m * (m + 1)) >> 1;
      const int total = ntop + (K + 1) * m;
      for (;;) {
        unsigned u = 0;
        if (lane == 0) u = atomicAdd(s_counter, 1u);
        u = __shfl_sync(0xffffffffu, u, 0);
        if ((int)u >= total) break;
        int I, J;
        if ((int)u < ntop) {
          int Ip = (int)((sqrtf(8.f * (float)u + 1.f) - 1.f) * 0.5f);
          while (((Ip + 1) * (Ip + 2) >> 1) <= (int)u) ++Ip;
          while (((Ip * (Ip + 1)) >> 1) > (int)u) --Ip;
          I = K + 1 + Ip;
          J = K + 1 + (int)u - ((Ip * (Ip + 1)) >> 1);
        } else {
          const int v = (int)u - ntop;
          I = Tn + v / m;
          J = K + 1 + v % m;
        }
        tile::tile_update(tile_at(I, J), tile_at(I, K), tile_at(J, K), lane);
      }
    }
    __syncthreads();
  }
  if (warp == 0 && lane == 0 && bad >= 0) report_error(status, THANOS_ERR_NOT_SPD, k0 + n - 1 - bad);
  // U22[i][j] = inv(L)[n-1-i][n-1-j] = identity row (n-1-j), column n-1-i
  for (int i = warp; i < n; i += DIAG_THREADS / 32) {
    for (int c4 = lane * 4; c4 < n; c4 += 128) {
      float u4[4];
      const int64_t o = (int64_t)(k0 + i) * b + k0 + c4;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int j = c4 + e;
        float u = 0.f;
        if (j >= i) {
          // (the factor V22 itself is not written back: nothing reads this block of V again)
          const int li = n - 1 - i, lj = n - 1 - j;  // lj <= li
          u = tile_at(Tn + (lj >> 4), li >> 4)[tile::elem_off(lj & 15, li & 15)];
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
  dim3 cg((unsigned)ceil_div(b, 4 * 256), (unsigned)b);
  copy_damped_upper_kernel<<<cg, 256, 0, stream>>>(H, w.V, b, w.lam);
  THANOS_CHECK_LAUNCH();
  THANOS_CUDA(cudaMemsetAsync(factor, 0, (size_t)plane * sizeof(float), stream));
  THANOS_CUDA(cudaMemsetAsync(w.Up, 0, 3 * (size_t)plane * sizeof(__nv_bfloat16), stream));
  THANOS_CUDA(cudaMemsetAsync(w.tc_status, 0, 16, stream));

  {
    static std::atomic<unsigned long long> done{0};
    THANOS_CUDA(ensure_max_dyn_smem(diag_block_kernel, DIAG_SMEM, done));
  }
  // ---- H_d = V V^T, panels from the last one backwards.  Full panels go in groups: a panel's
  //      own 128 columns first receive, in one product, what the earlier panels of its group
  //      owe them, and after the group's last panel a single product with K = 128 * (panels in
  //      the group) updates everything to the left -- the trailing matrix is read and written
  //      once per group instead of once per panel.
  auto diag_block = [&](int k0, int n) -> thanos_status_t {
    diag_block_kernel<<<1, DIAG_THREADS, DIAG_SMEM, stream>>>(w.V, factor, w.Up, plane, b, k0, n,
                                                              status_dev);
    THANOS_CHECK_LAUNCH();
    return THANOS_OK;
  };
  // V12 = A12 U22^T for the rows above the block at k0, written over A12 and as planes
  auto panel = [&](int k0, int n) -> thanos_status_t {
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
    return tc_gemm_split3(g, stream);
  };
  // V[0:M, c0:c0+N] -= P P[c0:c0+N, :]^T with P = V12 panel columns [kc, kc + K): c0 = 0, N = M is
  // the trailing update on the tiles that touch the upper triangle
  auto downdate = [&](int M, int c0, int N, int kc, int K, int upper) -> thanos_status_t {
    TcGemmArgs y;
    y.D = w.V + c0;
    y.ldd = b;
    y.A = w.Vp + kc;
    y.lda = b;
    y.a_plane = plane;
    y.B = w.Vp + (int64_t)c0 * b + kc;
    y.ldb = b;
    y.b_plane = plane;
    y.b_kmajor = 1;
    y.M = M;
    y.N = N;
    y.K = K;
    y.alpha = -1.f;
    y.accumulate = 1;
    y.upper_only = upper;
    y.status = w.tc_status;
    return tc_gemm_split3(y, stream);
  };
  for (int kb = nblk - 1; kb >= 0;) {
    const int k0 = kb * NB;
    const int n = (b - k0 < NB) ? b - k0 : NB;
    if (n < NB) {  // a ragged last panel goes alone
      THANOS_TRY(diag_block(k0, n));
      if (k0 == 0) break;
      THANOS_TRY(panel(k0, n));
      THANOS_TRY(downdate(k0, 0, k0, k0, n, 1));
      kb -= 1;
      continue;
    }
    int done = 0;
    bool finished = false;  // the group reached the first panel
    for (int j = 0; j < PANEL_GROUP; ++j) {
      const int kj = k0 - j * NB;
      // the panel's own columns first get what the group's earlier panels owe them
      if (j > 0) THANOS_TRY(downdate(kj + NB, kj, NB, kj + NB, j * NB, 0));
      THANOS_TRY(diag_block(kj, NB));
      if (kj == 0) {
        finished = true;
        break;
      }
      THANOS_TRY(panel(kj, NB));
      ++done;
    }
    if (finished) break;
    const int kl = k0 - (done - 1) * NB;  // first column of the group
    THANOS_TRY(downdate(kl, 0, kl, kl, done * NB, 1));
    kb -= done;
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
