// 16 x 16 fp32 tiles in shared memory for the tile Cholesky kernels: layout, the diagonal-tile
// factorisation by one warp and the tile update C -= A B^T by one warp.
#pragma once

#include "common.cuh"

namespace thanos {
namespace tile {

constexpr unsigned FULL_MASK = 0xffffffffu;

// A tile is 256 floats, row-major in 16-byte chunks; chunk c of row r sits at chunk position
// c ^ swizzle(r) with swizzle = (bit 1 of r, bit 2 of r), which keeps the access patterns of the
// functions below, and the accumulator fragments of mma.m16n8k16, free of bank conflicts.
__device__ __forceinline__ int chunk_swizzle(int r) { return (r & 2) | ((r >> 2) & 1); }
__device__ __forceinline__ int chunk_off(int r, int c) { return (r << 4) + ((c ^ chunk_swizzle(r)) << 2); }
__device__ __forceinline__ int elem_off(int r, int k) { return chunk_off(r, k >> 2) + (k & 3); }

// Cholesky of a diagonal tile by one warp: lane r < 16 holds row r.  Columns col0 + j >= n (a
// right-hand-side row, identity padding) get pivot 1.  invd[col0 + j] = 1 / l_jj.  Returns the
// first column with a non-positive pivot, -1 if there is none.  NEWTON refines the reciprocal
// square root by one Newton step.
template <bool NEWTON>
__device__ __forceinline__ int factor_diag_tile(float* __restrict__ Tt, float* __restrict__ invd,
                                                int col0, int n, int lane) {
  const int r = lane & 15;
  float a[16];
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    const float4 v = *reinterpret_cast<const float4*>(Tt + chunk_off(r, c));
    a[4 * c] = v.x; a[4 * c + 1] = v.y; a[4 * c + 2] = v.z; a[4 * c + 3] = v.w;
  }
  int bad = -1;
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    float dj = __shfl_sync(FULL_MASK, a[j], j);
    if (col0 + j < n) {
      if (!(dj > 0.f) || !isfinite(dj)) {
        if (bad < 0) bad = col0 + j;
        dj = 1.f;
      }
    } else {
      dj = 1.f;
    }
    float rinv = rsqrtf(dj);
    if (NEWTON) rinv = rinv * fmaf(-0.5f * dj, rinv * rinv, 1.5f);
    if (lane == 0) invd[col0 + j] = rinv;
    a[j] *= rinv;
#pragma unroll
    for (int v = j + 1; v < 16; ++v) {
      const float lvj = __shfl_sync(FULL_MASK, a[j], v);
      a[v] = fmaf(-a[j], lvj, a[v]);
    }
  }
  if (lane < 16) {
#pragma unroll
    for (int c = 0; c < 4; ++c)
      *reinterpret_cast<float4*>(Tt + chunk_off(r, c)) =
          make_float4(a[4 * c], a[4 * c + 1], a[4 * c + 2], a[4 * c + 3]);
  }
  __syncwarp();
  return bad;
}

// C -= A B^T for 16 x 16 tiles by one warp: lane (lr, lc) owns rows lr, lr + 8 and columns
// lc, lc + 4, lc + 8, lc + 12.
__device__ __forceinline__ void tile_update(float* __restrict__ Ct, const float* __restrict__ At,
                                            const float* __restrict__ Bt, int lane) {
  const int lr = lane >> 2, lc = lane & 3;
  float acc[2][4];
#pragma unroll
  for (int i = 0; i < 4; ++i) acc[0][i] = acc[1][i] = 0.f;
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    const float4 a0 = *reinterpret_cast<const float4*>(At + chunk_off(lr, c));
    const float4 a1 = *reinterpret_cast<const float4*>(At + chunk_off(lr + 8, c));
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float4 bv = *reinterpret_cast<const float4*>(Bt + chunk_off(lc + 4 * i, c));
      acc[0][i] = fmaf(a0.x, bv.x, acc[0][i]);
      acc[0][i] = fmaf(a0.y, bv.y, acc[0][i]);
      acc[0][i] = fmaf(a0.z, bv.z, acc[0][i]);
      acc[0][i] = fmaf(a0.w, bv.w, acc[0][i]);
      acc[1][i] = fmaf(a1.x, bv.x, acc[1][i]);
      acc[1][i] = fmaf(a1.y, bv.y, acc[1][i]);
      acc[1][i] = fmaf(a1.z, bv.z, acc[1][i]);
      acc[1][i] = fmaf(a1.w, bv.w, acc[1][i]);
    }
  }
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int r = lr + 8 * h;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float* p = Ct + chunk_off(r, i) + lc;  // column lc + 4 i: chunk i, element lc
      *p -= acc[h][i];
    }
  }
}

// The rows of a panel below (or beside) a factored diagonal tile Lk: x L_k^T = a for one row
// of 16 entries held by one thread; invd = 1 / diag(L_k) for the tile's 16 columns.
__device__ __forceinline__ void panel_row_solve(float* arow_tile, int r, const float* Lk,
                                                const float* invd16) {
  float x[16];
#pragma unroll
  for (int cc = 0; cc < 4; ++cc) {
    const float4 v = *reinterpret_cast<const float4*>(arow_tile + chunk_off(r, cc));
    x[4 * cc] = v.x; x[4 * cc + 1] = v.y; x[4 * cc + 2] = v.z; x[4 * cc + 3] = v.w;
  }
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    float l[16];
#pragma unroll
    for (int cc = 0; cc <= ((j - 1) >> 2) && j > 0; ++cc) {
      const float4 v = *reinterpret_cast<const float4*>(Lk + chunk_off(j, cc));
      l[4 * cc] = v.x; l[4 * cc + 1] = v.y; l[4 * cc + 2] = v.z; l[4 * cc + 3] = v.w;
    }
    float acc = x[j];
#pragma unroll
    for (int mm = 0; mm < j; ++mm) acc = fmaf(-x[mm], l[mm], acc);
    x[j] = acc * invd16[j];
  }
#pragma unroll
  for (int cc = 0; cc < 4; ++cc)
    *reinterpret_cast<float4*>(arow_tile + chunk_off(r, cc)) =
        make_float4(x[4 * cc], x[4 * cc + 1], x[4 * cc + 2], x[4 * cc + 3]);
}

}  // namespace tile
}  // namespace thanos
