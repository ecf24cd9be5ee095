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

// ---- tile products on the tensor cores (mma.sync m16n8k16): fp32 tiles are split into three
// bf16 planes in registers (24 significant bits) and six plane products are accumulated in fp32.
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0,
                                               uint32_t b1) {
  // no side effects beyond its outputs: not volatile, so that independent chains interleave
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// (x0, x1) -> three words of two bf16 each (x0 in the low half): x = p0 + p1 + p2 to 24 bits
__device__ __forceinline__ void split_pair(float x0, float x1, uint32_t& p0, uint32_t& p1,
                                           uint32_t& p2) {
  __nv_bfloat162 h = __floats2bfloat162_rn(x0, x1);
  p0 = *reinterpret_cast<const uint32_t*>(&h);
  x0 -= __uint_as_float(p0 << 16);
  x1 -= __uint_as_float(p0 & 0xffff0000u);
  h = __floats2bfloat162_rn(x0, x1);
  p1 = *reinterpret_cast<const uint32_t*>(&h);
  x0 -= __uint_as_float(p1 << 16);
  x1 -= __uint_as_float(p1 & 0xffff0000u);
  h = __floats2bfloat162_rn(x0, x1);
  p2 = *reinterpret_cast<const uint32_t*>(&h);
}

// Fragment of a 16 x 16 panel tile P for mma.m16n8k16 (g = lane / 4, t = lane % 4): word 0 rows g,
// columns 2t, 2t + 1; word 1 row g + 8; words 2, 3 the same rows, columns 2t + 8, 2t + 9.  As the A
// operand (P itself) all four words are used; as the B operand (P^T) half h of the 8-wide column
// blocks takes words h and h + 2.
struct PanelFrag {
  uint32_t w[3][4];
};
// Offsets of a lane's four fragment words inside any tile (they depend on the lane only): word
// 2 h' + h'' is row g + 8 h'', columns 2t + 8 h' -- also the lane's accumulator entries of column
// half h'.
struct FragOff {
  int o[4];
};
__device__ __forceinline__ FragOff make_frag_off(int g, int t) {
  FragOff f;
  f.o[0] = elem_off(g, 2 * t);
  f.o[1] = elem_off(g + 8, 2 * t);
  f.o[2] = elem_off(g, 2 * t + 8);
  f.o[3] = elem_off(g + 8, 2 * t + 8);
  return f;
}
__device__ __forceinline__ void load_panel_frag(const float* __restrict__ Tt, const FragOff& fo,
                                                PanelFrag& f) {
  const float2 v0 = *reinterpret_cast<const float2*>(Tt + fo.o[0]);
  const float2 v1 = *reinterpret_cast<const float2*>(Tt + fo.o[1]);
  const float2 v2 = *reinterpret_cast<const float2*>(Tt + fo.o[2]);
  const float2 v3 = *reinterpret_cast<const float2*>(Tt + fo.o[3]);
  split_pair(v0.x, v0.y, f.w[0][0], f.w[1][0], f.w[2][0]);
  split_pair(v1.x, v1.y, f.w[0][1], f.w[1][1], f.w[2][1]);
  split_pair(v2.x, v2.y, f.w[0][2], f.w[1][2], f.w[2][2]);
  split_pair(v3.x, v3.y, f.w[0][3], f.w[1][3], f.w[2][3]);
}

// acc[h] += P_a P_b^T (the two 8-column halves h) from the six plane products, smallest first
__device__ __forceinline__ void frag_product(float (&acc)[2][4], const PanelFrag& fa,
                                             const PanelFrag& fb) {
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    mma_bf16_16816(acc[h], fa.w[1], fb.w[1][h], fb.w[1][h + 2]);  // m m
    mma_bf16_16816(acc[h], fa.w[2], fb.w[0][h], fb.w[0][h + 2]);  // l h
    mma_bf16_16816(acc[h], fa.w[0], fb.w[2][h], fb.w[2][h + 2]);  // h l
    mma_bf16_16816(acc[h], fa.w[1], fb.w[0][h], fb.w[0][h + 2]);  // m h
    mma_bf16_16816(acc[h], fa.w[0], fb.w[1][h], fb.w[1][h + 2]);  // h m
    mma_bf16_16816(acc[h], fa.w[0], fb.w[0][h], fb.w[0][h + 2]);  // h h
  }
}

// C -= acc for one target tile (accumulator layout: rows g, g + 8, columns 8 h + 2 t, + 1)
__device__ __forceinline__ void tile_subtract(float* __restrict__ Ct, const float (&acc)[2][4],
                                              const FragOff& fo) {
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    float2* c0 = reinterpret_cast<float2*>(Ct + fo.o[2 * h]);
    float2* c1 = reinterpret_cast<float2*>(Ct + fo.o[2 * h + 1]);
    float2 u0 = *c0, u1 = *c1;
    u0.x -= acc[h][0];
    u0.y -= acc[h][1];
    u1.x -= acc[h][2];
    u1.y -= acc[h][3];
    *c0 = u0;
    *c1 = u1;
  }
}

}  // namespace tile
}  // namespace thanos
