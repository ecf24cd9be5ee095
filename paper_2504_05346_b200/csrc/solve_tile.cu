// Per-row constrained solve of one block step (Eqs. 5-8) for systems of up to 64 unknowns: one warp
// per row, tile Cholesky whose panel and trailing products run on the tensor cores.
//
// Same mathematics as solve.cu (direct form on G for rows with |q| <= |k|, complement form on S
// otherwise).  The gathered matrix lives in shared memory as the lower triangle of 16 x 16 fp32
// tiles (tile_ops.cuh).  Per tile column K the warp
//   factors the diagonal tile with warp shuffles -- lanes 0..15 hold its rows, lanes 16..31 the
//   rows of the identity, and the same column operations leave L_KK in the former and L_KK^{-T}
//   in the latter (kept in the unused upper triangle of the tile);
//   forms the panel below it as a product, L_IK = A_IK L_KK^{-T};
//   and subtracts L_IK L_JK^T from every trailing tile.
// The products use mma.sync m16n8k16: fp32 tiles are split into three bf16 planes in registers
// (24 significant bits), six plane products are accumulated in fp32; the accumulator layout of a
// panel product is the A-operand layout of the trailing product, so a panel tile goes from one to
// the other without leaving the registers.  The right-hand side is a vector of its own; with the
// inverses of the diagonal tiles both substitutions are 16 x 16 matrix-vector products per tile
// row, and the only serial chains left are the four diagonal factorisations.
#include "common.cuh"
#include "tile_ops.cuh"

namespace thanos {

namespace {

using tile::chunk_off;
using tile::elem_off;
using tile::FragOff;
using tile::PanelFrag;
using tile::frag_product;
using tile::load_panel_frag;
using tile::make_frag_off;
using tile::mma_bf16_16816;
using tile::split_pair;
using tile::tile_subtract;

constexpr unsigned FULL = 0xffffffffu;
constexpr int TILE_T_MAX = 4;  // tile rows: systems of up to 64 unknowns

__device__ __forceinline__ int tbase(int I, int J) { return (((I * (I + 1)) >> 1) + J) << 8; }

struct TileSolveLayout {
  int tiles_floats;
  int per_warp_bytes;
};

__host__ __device__ inline TileSolveLayout tile_solve_layout(int Bw, int T) {
  TileSolveLayout L;
  L.tiles_floats = (T * (T + 1) / 2) * 256;
  // tiles, invd[16 T], yv[16 T + 16], wblk[Bw], dvec[Bw], two index lists of Bw + 16 shorts
  const int bytes = 4 * (L.tiles_floats + 16 * T + 16 * T + 16 + 2 * Bw) + 2 * 2 * (Bw + 16);
  L.per_warp_bytes = (bytes + 15) & ~15;
  return L;
}


// Panel tile as a product: L_IK = A_IK L_KK^{-T} (fa: fragment of A_IK, fl: fragment of
// L_KK^{-1}).  The result is stored over A_IK and returned as the fragment for the trailing
// updates (the accumulator layout is the A-operand layout).
__device__ __forceinline__ void panel_product(float* __restrict__ Tt, const PanelFrag& fa,
                                              const PanelFrag& fl, const FragOff& fo,
                                              PanelFrag& out) {
  float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
  frag_product(acc, fa, fl);
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    *reinterpret_cast<float2*>(Tt + fo.o[2 * h]) = make_float2(acc[h][0], acc[h][1]);
    *reinterpret_cast<float2*>(Tt + fo.o[2 * h + 1]) = make_float2(acc[h][2], acc[h][3]);
    split_pair(acc[h][0], acc[h][1], out.w[0][2 * h], out.w[1][2 * h], out.w[2][2 * h]);
    split_pair(acc[h][2], acc[h][3], out.w[0][2 * h + 1], out.w[1][2 * h + 1], out.w[2][2 * h + 1]);
  }
}

// Cholesky of a diagonal tile together with the inverse of its factor.  Lanes 0..15 hold the rows
// of A_KK, lanes 16..31 the rows of the identity; the column operations of the factorisation
// (scale column j, subtract its multiples from the columns to the right) turn [A_KK; I] into
// [L; L^{-T}].  Every lane also carries its own diagonal entry, so the pivot of the next column
// does not wait for the updates of the others.  Stored: L in the lower triangle and diagonal of
// the tile, the strict upper triangle of L^{-T} above it, 1 / l_jj (the diagonal of L^{-1}) in
// invd.  Columns col0 + j >= n (identity padding) get pivot 1.  Returns whether a pivot was not
// positive and finite.  `ident` is an identity tile in the tile layout, rc / doff the offsets of
// the chunks and of the diagonal entry of row lane % 16.
__device__ __forceinline__ bool factor_diag_tile_inv(float* __restrict__ Tt,
                                                     const float* __restrict__ ident,
                                                     float* __restrict__ invd, int col0, int n,
                                                     int lane, const int (&rc)[4], int doff) {
  const int r = lane & 15;
  const bool top = lane < 16;
  // rows of the tile for lanes 0..15, rows of the identity (same tile layout) for lanes 16..31
  const float* src = top ? Tt : ident;
  float a[16];
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    const float4 v = *reinterpret_cast<const float4*>(src + rc[c]);
    a[4 * c] = v.x; a[4 * c + 1] = v.y; a[4 * c + 2] = v.z; a[4 * c + 3] = v.w;
  }
  float diag = Tt[doff];
  const int nlive = n - col0;  // columns beyond it are identity padding
  bool bad = false;
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    float dj = __shfl_sync(FULL, diag, j);
    const bool okp = dj > 0.f && dj < 3.0e38f;  // positive and finite
    if (j < nlive && !okp) bad = true;
    dj = (j < nlive && okp) ? dj : 1.f;
    const float rinv = rsqrtf(dj);
    if (lane == 0) invd[col0 + j] = rinv;
    a[j] *= rinv;
    diag = fmaf(-a[j], a[j], diag);  // meaningful for the rows below j, whose pivots come later
#pragma unroll
    for (int v = j + 1; v < 16; ++v) {
      const float lvj = __shfl_sync(FULL, a[j], v);
      a[v] = fmaf(-a[j], lvj, a[v]);
    }
  }
  // row r of the tile: columns <= r from the upper half-warp (L), columns > r from the lower
  // half-warp (L^{-T})
#pragma unroll
  for (int cidx = 0; cidx < 16; ++cidx) {
    if (top ? (cidx <= r) : (cidx > r)) Tt[rc[cidx >> 2] + (cidx & 3)] = a[cidx];
  }
  __syncwarp();
  return bad;
}

// Fragment of L_KK^{-1} (lower triangular) from a factored diagonal tile: entry (i, j), j < i, is
// stored transposed at (j, i); the diagonal is invd.  Where a lane's eight entries sit depends on
// the lane only: `off` holds the tile offsets of the entries below the diagonal, bit e of `below`
// / `ondiag` says which kind entry e is (entry 2 w + e: row g + 8 (w & 1), column
// 2t + 8 (w >> 1) + e).
struct InvFragOff {
  int off[8];
  unsigned below, ondiag;
};
__device__ __forceinline__ InvFragOff make_inv_frag_off(int g, int t) {
  InvFragOff f;
  f.below = f.ondiag = 0;
#pragma unroll
  for (int w = 0; w < 4; ++w) {
    const int row = g + 8 * (w & 1);
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int col = 2 * t + 8 * (w >> 1) + e;
      f.off[2 * w + e] = col < row ? elem_off(col, row) : 0;
      if (col < row) f.below |= 1u << (2 * w + e);
      if (col == row) f.ondiag |= 1u << (2 * w + e);
    }
  }
  return f;
}
__device__ __forceinline__ void load_inverse_frag(const float* __restrict__ Tt,
                                                  const float* __restrict__ invd16, int g,
                                                  const InvFragOff& io, PanelFrag& f) {
  const float d0 = invd16[g], d1 = invd16[g + 8];
  float v[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const float x = Tt[io.off[i]];  // offset 0 (a valid entry) where the value is not used
    v[i] = (io.below >> i) & 1u ? x : ((io.ondiag >> i) & 1u ? ((i >> 1) & 1 ? d1 : d0) : 0.f);
  }
#pragma unroll
  for (int w = 0; w < 4; ++w) split_pair(v[2 * w], v[2 * w + 1], f.w[0][w], f.w[1][w], f.w[2][w]);
}

// One warp per row; the arguments and the split of the CTAs between the two kinds of rows are
// those of solve_rows_fast_kernel (solve.cu).  `tiles` is the number of tile rows the launch
// provides room for; a row uses ceil(n / 16) of them.
__global__ void __launch_bounds__(32 * 16)
solve_rows_tile_kernel(float* __restrict__ Wc, const uint8_t* __restrict__ mask,
                       const float* __restrict__ Gm, const float* __restrict__ Sm, int ld_mat,
                       __nv_bfloat16* __restrict__ D, int64_t dplane, int c, int b, int j1, int Bw,
                       int ldd, int tiles, const int* __restrict__ row_lists,
                       const unsigned* __restrict__ list_counts, int fixed_kind, int report_max_s,
                       thanos_stats_t* stats) {
  extern __shared__ __align__(16) unsigned char dyn[];
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int warps = blockDim.x >> 5;
  const TileSolveLayout lay = tile_solve_layout(Bw, tiles);
  unsigned char* wbase = dyn + (size_t)warp * lay.per_warp_bytes;
  float* A = reinterpret_cast<float*>(wbase);
  float* invd = A + lay.tiles_floats;
  float* yv = invd + 16 * tiles;
  float* wblk = yv + 16 * tiles + 16;
  float* dvec = wblk + Bw;
  unsigned short* qlist = reinterpret_cast<unsigned short*>(dvec + Bw);
  unsigned short* klist = qlist + Bw + 16;
  const int g = lane >> 2, t4 = lane & 3;
  const FragOff fo = make_frag_off(g, t4);
  const InvFragOff io = make_inv_frag_off(g, t4);
  // chunk offsets and diagonal entry of tile row lane % 16
  int rc[4];
#pragma unroll
  for (int cc = 0; cc < 4; ++cc) rc[cc] = chunk_off(lane & 15, cc);
  const int doff = elem_off(lane & 15, lane & 15);
  // an identity tile (the lower half-warp of a diagonal factorisation starts from its rows)
  __shared__ __align__(16) float s_ident[256];
  for (int e = threadIdx.x; e < 256; e += blockDim.x) s_ident[elem_off(e >> 4, e & 15)] = (e >> 4) == (e & 15) ? 1.f : 0.f;
  __syncthreads();
  // forward substitution: lane (l = lane % 16, half = lane / 16) reads column l of the upper
  // triangle of a diagonal tile, rows 8 half .. 8 half + 7
  int fwd_off[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) fwd_off[e] = elem_off(8 * (lane >> 4) + e, lane & 15);
  // gather: lane (r0 = lane / 16, k = lane % 16) fills rows r0 + 2 h of column k of a tile
  int gofs[8];
#pragma unroll
  for (int h = 0; h < 8; ++h) gofs[h] = elem_off((lane >> 4) + 2 * h, lane & 15);

  int cnt[2];
  if (row_lists) {
    cnt[0] = (int)list_counts[0];
    cnt[1] = (int)list_counts[1];
  } else {
    cnt[fixed_kind] = c;
    cnt[fixed_kind ^ 1] = 0;
  }
  const int nctas = gridDim.x;
  int n1 = 0;  // CTAs [0, nctas - n1) serve kind 0, the rest kind 1
  if (cnt[1] > 0) {
    if (cnt[0] == 0) {
      n1 = nctas;
    } else {
      n1 = (int)(((long long)nctas * cnt[1] + (cnt[0] + cnt[1]) / 2) / (cnt[0] + cnt[1]));
      if (n1 < 1) n1 = 1;
      if (n1 > nctas - 1) n1 = nctas - 1;
    }
  }
  const bool both_here = nctas == 1 && cnt[0] > 0 && cnt[1] > 0;
  const unsigned lt = (1u << lane) - 1u;

  for (int pass = 0; pass < (both_here ? 2 : 1); ++pass) {
    int kind, my_index, my_ctas;
    if (both_here) {
      kind = pass;
      my_index = 0;
      my_ctas = 1;
    } else if ((int)blockIdx.x < nctas - n1) {
      kind = 0;
      my_index = blockIdx.x;
      my_ctas = nctas - n1;
    } else {
      kind = 1;
      my_index = blockIdx.x - (nctas - n1);
      my_ctas = n1;
    }
    if (cnt[kind] == 0) continue;  // CTA-uniform
    const bool kpath = kind == 1;
    // G / S are read from global memory (64 KB at B = 128: they stay in L2); a shared copy
    // would cost three of sixteen warps and buys no throughput
    const float* M = kpath ? Sm : Gm;
    const int ldm = ld_mat;
    const int* rlist = row_lists ? row_lists + (size_t)kind * c : nullptr;

    for (int li = my_index * warps + warp; li < cnt[kind]; li += my_ctas * warps) {
      const int row = rlist ? rlist[li] : li;
      const uint8_t* mrow = mask + (int64_t)row * b + j1;
      float* wrow = Wc + (int64_t)row * b + j1;
      // ---- q = phi(mask row) and its complement k, both ascending
      int s = 0, t = 0;
      for (int base = 0; base < Bw; base += 128) {
        uint8_t mv[4];
        float wv[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int jj = base + 32 * u + lane;
          mv[u] = (jj < Bw) ? mrow[jj] : (uint8_t)2;
          wv[u] = (jj < Bw) ? wrow[jj] : 0.f;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int jj = base + 32 * u + lane;
          const bool mb = mv[u] == 1;
          const bool kb = mv[u] == 0;
          const unsigned bq = __ballot_sync(FULL, mb);
          const unsigned bk = __ballot_sync(FULL, kb);
          if (mb) qlist[s + __popc(bq & lt)] = (unsigned short)jj;
          if (kb) klist[t + __popc(bk & lt)] = (unsigned short)jj;
          if (jj < Bw) wblk[jj] = wv[u];
          s += __popc(bq);
          t += __popc(bk);
        }
      }
      if (s == 0) {  // nothing removed: the row is not touched in this block
        for (int jj = lane; jj < Bw; jj += 32) store_split3(D + (int64_t)row * ldd + jj, dplane, 0.f);
        __syncwarp();
        continue;
      }
      if (report_max_s && row == 0 && lane == 0) atomicMax(&stats->max_s, s);
      const int n = kpath ? t : s;    // unknowns of this row's system
      const int no = kpath ? s : t;   // size of the other set
      unsigned short* sel = kpath ? klist : qlist;
      unsigned short* oth = kpath ? qlist : klist;
      if (lane < 16) {
        sel[n + lane] = 0;
        oth[no + lane] = 0;
      }
      const int T = (n + 15) >> 4;
      if (n == 0) {  // every weight of the block is removed: delta = -w, nothing to solve
        for (int jj = lane; jj < Bw; jj += 32) {
          const float d = -wblk[jj];
          wrow[jj] = 0.f;
          store_split3(D + (int64_t)row * ldd + jj, dplane, d);
        }
        __syncwarp();
        continue;
      }
      if ((s > t) != kpath || T > tiles) {
        // cannot happen for lists and launch sizes made by this library
        if (lane == 0) report_error(&stats->status, THANOS_ERR_SHAPE, row);
        __syncwarp();
        continue;
      }
      __syncwarp();
      // ---- right-hand side: w_q (direct form) or g_e = sum_a w[q_a] S[q_a, k_e] (complement),
      //      zero beyond n
      if (!kpath) {
        for (int e = lane; e < 16 * T; e += 32) yv[e] = e < n ? wblk[sel[e]] : 0.f;
      } else {
        // the removed weights in list order, zero-padded to a multiple of four
        for (int a = lane; a < ((no + 3) & ~3); a += 32) dvec[a] = a < no ? wblk[oth[a]] : 0.f;
        __syncwarp();
        for (int e0 = 0; e0 < 16 * T; e0 += 32) {
          const int e = e0 + lane;
          const int col = (e < n) ? (int)sel[e] : 0;
          float g0 = 0.f, g1 = 0.f;
          for (int a = 0; a < no; a += 4) {
            const ushort4 ix = *reinterpret_cast<const ushort4*>(oth + a);
            const float4 wq = *reinterpret_cast<const float4*>(dvec + a);
            g0 = fmaf(wq.x, M[(int)ix.x * ldm + col], g0);
            g1 = fmaf(wq.y, M[(int)ix.y * ldm + col], g1);
            g0 = fmaf(wq.z, M[(int)ix.z * ldm + col], g0);
            g1 = fmaf(wq.w, M[(int)ix.w * ldm + col], g1);
          }
          if (e < 16 * T) yv[e] = e < n ? g0 + g1 : 0.f;
        }
        __syncwarp();
      }
      // ---- gather the lower triangle of M[sel, sel] into tiles, identity beyond n
      {
        const int r0 = lane >> 4, k = lane & 15;
        for (int I = 0; I < T; ++I) {
          const bool rows_in = 16 * I + 16 <= n;  // warp-uniform: every row of the tile row exists
          int rowoff[8];
#pragma unroll
          for (int h = 0; h < 8; ++h) {
            const int i = 16 * I + r0 + 2 * h;
            rowoff[h] = (rows_in || i < n) ? (int)sel[i] * ldm : -1;
          }
          for (int J = 0; J <= I; ++J) {
            const int j = 16 * J + k;
            float* Tt = A + tbase(I, J);
            float v[8];
            if (rows_in) {  // columns j <= i < n as well
              const float* Mc = M + (int)sel[j];
#pragma unroll
              for (int h = 0; h < 8; ++h) v[h] = Mc[rowoff[h]];
            } else {
              const int cj = j < n ? (int)sel[j] : -1;
#pragma unroll
              for (int h = 0; h < 8; ++h) {
                const int i = 16 * I + r0 + 2 * h;
                v[h] = (rowoff[h] >= 0 && cj >= 0) ? M[rowoff[h] + cj] : (i == j ? 1.f : 0.f);
              }
            }
#pragma unroll
            for (int h = 0; h < 8; ++h) Tt[gofs[h]] = v[h];
          }
        }
      }
      __syncwarp();

      // ---- right-looking tile Cholesky
      bool bad = false;
      for (int K = 0; K < T; ++K) {
        float* Lk = A + tbase(K, K);
        bad |= factor_diag_tile_inv(Lk, s_ident, invd, 16 * K, n, lane, rc, doff);
        const int m = T - K - 1;  // tile rows below the diagonal tile (warp-uniform, <= 3)
        if (m == 0) break;
        // panel tiles as products with the inverse of the diagonal factor
        PanelFrag fl, f0, f1, f2;
        load_inverse_frag(Lk, invd + 16 * K, g, io, fl);
        {
          PanelFrag fa;
          load_panel_frag(A + tbase(K + 1, K), fo, fa);
          panel_product(A + tbase(K + 1, K), fa, fl, fo, f0);
          if (m > 1) {
            load_panel_frag(A + tbase(K + 2, K), fo, fa);
            panel_product(A + tbase(K + 2, K), fa, fl, fo, f1);
          }
          if (m > 2) {
            load_panel_frag(A + tbase(K + 3, K), fo, fa);
            panel_product(A + tbase(K + 3, K), fa, fl, fo, f2);
          }
        }
        // trailing tiles, one tile row at a time (its products are independent chains)
        {
          float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
          frag_product(acc, f0, f0);
          tile_subtract(A + tbase(K + 1, K + 1), acc, fo);
        }
        if (m > 1) {
          float a0[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
          float a1[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
          frag_product(a0, f1, f0);
          frag_product(a1, f1, f1);
          tile_subtract(A + tbase(K + 2, K + 1), a0, fo);
          tile_subtract(A + tbase(K + 2, K + 2), a1, fo);
        }
        if (m > 2) {
          float a0[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
          float a1[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
          float a2[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
          frag_product(a0, f2, f0);
          frag_product(a1, f2, f1);
          frag_product(a2, f2, f2);
          tile_subtract(A + tbase(K + 3, K + 1), a0, fo);
          tile_subtract(A + tbase(K + 3, K + 2), a1, fo);
          tile_subtract(A + tbase(K + 3, K + 3), a2, fo);
        }
        __syncwarp();
      }
      if (bad) {
        if (lane == 0) report_error(&stats->status, THANOS_ERR_NOT_SPD, row);
        for (int jj = lane; jj < Bw; jj += 32) store_split3(D + (int64_t)row * ldd + jj, dplane, 0.f);
        __syncwarp();
        continue;
      }

      const int l16 = lane & 15, hh = lane >> 4;
      // ---- forward substitution L y = rhs by tile rows: y_I = L_II^{-1} (rhs_I - sum_J L_IJ y_J);
      //      lanes l and l + 16 share row l (columns 0..7 and 8..15 of every tile)
      for (int I = 0; I < T; ++I) {
        if (I > 0) {
          float acc = 0.f;
          for (int J = 0; J < I; ++J) {
            const float* Lt = A + tbase(I, J);
            const float4 a0 = *reinterpret_cast<const float4*>(Lt + (hh ? rc[2] : rc[0]));
            const float4 a1 = *reinterpret_cast<const float4*>(Lt + (hh ? rc[3] : rc[1]));
            const float4 y0 = *reinterpret_cast<const float4*>(yv + 16 * J + 8 * hh);
            const float4 y1 = *reinterpret_cast<const float4*>(yv + 16 * J + 8 * hh + 4);
            acc = fmaf(a0.x, y0.x, acc); acc = fmaf(a0.y, y0.y, acc);
            acc = fmaf(a0.z, y0.z, acc); acc = fmaf(a0.w, y0.w, acc);
            acc = fmaf(a1.x, y1.x, acc); acc = fmaf(a1.y, y1.y, acc);
            acc = fmaf(a1.z, y1.z, acc); acc = fmaf(a1.w, y1.w, acc);
          }
          acc += __shfl_xor_sync(FULL, acc, 16);
          __syncwarp();
          if (lane < 16) yv[16 * I + lane] -= acc;
          __syncwarp();
        }
        // y = L_II^{-1} v: entry (l, c), c < l, of the inverse sits at (c, l) of the tile
        const float* Lk = A + tbase(I, I);
        const float4 v0 = *reinterpret_cast<const float4*>(yv + 16 * I + 8 * hh);
        const float4 v1 = *reinterpret_cast<const float4*>(yv + 16 * I + 8 * hh + 4);
        const float vv[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
        float acc = 0.f;
        const float dl = invd[16 * I + l16];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const int cidx = 8 * hh + e;
          const float x = Lk[fwd_off[e]];  // entries on or below the diagonal are not used
          acc = fmaf(cidx < l16 ? x : (cidx == l16 ? dl : 0.f), vv[e], acc);
        }
        acc += __shfl_xor_sync(FULL, acc, 16);
        __syncwarp();
        if (lane < 16) yv[16 * I + lane] = acc;
        __syncwarp();
      }
      // ---- back substitution L^T x = y from the bottom: x_K = L_KK^{-T} y_K, then the rows above
      //      lose L_KJ^T x_K
      for (int Kb = T - 1; Kb >= 0; --Kb) {
        const float* Lk = A + tbase(Kb, Kb);
        {
          // row l of L^{-T}: columns > l in the tile's upper triangle, the diagonal in invd
          const float4 a0 = *reinterpret_cast<const float4*>(Lk + (hh ? rc[2] : rc[0]));
          const float4 a1 = *reinterpret_cast<const float4*>(Lk + (hh ? rc[3] : rc[1]));
          const float4 v0 = *reinterpret_cast<const float4*>(yv + 16 * Kb + 8 * hh);
          const float4 v1 = *reinterpret_cast<const float4*>(yv + 16 * Kb + 8 * hh + 4);
          const float aa[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
          const float vv[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
          const float dl = invd[16 * Kb + l16];
          float acc = 0.f;
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            const int cidx = 8 * hh + e;
            const float x = cidx > l16 ? aa[e] : (cidx == l16 ? dl : 0.f);
            acc = fmaf(x, vv[e], acc);
          }
          acc += __shfl_xor_sync(FULL, acc, 16);
          __syncwarp();
          if (lane < 16) yv[16 * Kb + lane] = acc;
          __syncwarp();
        }
        // earlier unknowns: y_k -= sum_w L[16 Kb + w][k] x_w
        for (int k = lane; k < 16 * Kb; k += 32) {
          const float* Lt = A + tbase(Kb, k >> 4);
          const int kk = k & 15;
          float acc = 0.f;
#pragma unroll
          for (int w = 0; w < 16; ++w) acc = fmaf(Lt[elem_off(w, kk)], yv[16 * Kb + w], acc);
          yv[k] -= acc;
        }
        __syncwarp();
      }

      // ---- delta over the block
      for (int a = lane; a < s; a += 32) dvec[qlist[a]] = -wblk[qlist[a]];
      if (kpath) {
        for (int e = lane; e < n; e += 32) dvec[sel[e]] = yv[e];
      } else {
        // delta_k = -sum_a lambda_a G[q_a, k_e]   (yv is zero beyond n)
        for (int e0 = 0; e0 < no; e0 += 32) {
          const int e = e0 + lane;
          const int col = (e < no) ? (int)oth[e] : 0;
          float g0 = 0.f, g1 = 0.f;
          for (int a = 0; a < n; a += 4) {
            const ushort4 ix = *reinterpret_cast<const ushort4*>(sel + a);
            const float4 xv = *reinterpret_cast<const float4*>(yv + a);
            g0 = fmaf(xv.x, M[(int)ix.x * ldm + col], g0);
            g1 = fmaf(xv.y, M[(int)ix.y * ldm + col], g1);
            g0 = fmaf(xv.z, M[(int)ix.z * ldm + col], g0);
            g1 = fmaf(xv.w, M[(int)ix.w * ldm + col], g1);
          }
          if (e < no) dvec[col] = -(g0 + g1);
        }
      }
      __syncwarp();
      for (int jj = lane; jj < Bw; jj += 32) {
        const float d = dvec[jj];
        const bool removed = mrow[jj] != 0;
        wrow[jj] = removed ? 0.f : wblk[jj] + d;
        store_split3(D + (int64_t)row * ldd + jj, dplane, d);
      }
      __syncwarp();
    }
  }
}

constexpr size_t TILE_SMEM_BUDGET = 227 * 1024;
constexpr int TILE_MAX_WARPS = 16;

}  // namespace

int tile_solve_max_unknowns() { return 16 * TILE_T_MAX; }

// Same contract as launch_fast of solve.cu; n_max <= 64.
thanos_status_t launch_tile_solve(float* Wc, const uint8_t* mask, const float* G, const float* S,
                                  int ld_mat, __nv_bfloat16* D, int64_t dplane, int c, int b,
                                  int j1, int Bw, int ldd, int n_max, const int* row_lists,
                                  const unsigned* list_counts, int fixed_kind, int report_max_s,
                                  thanos_stats_t* stats, cudaStream_t stream) {
  const int T = (n_max + 15) / 16 < 1 ? 1 : (n_max + 15) / 16;
  if (T > TILE_T_MAX) return THANOS_ERR_SHAPE;
  // The kernel is bound by instruction issue, not by latency: an SM finishes a row every ~3.9 k
  // cycles whether 13, 16 or 18 warps share it (measured), so a row takes (warps) x 3.9 k cycles and
  // a launch lasts (rows per warp, rounded up) x (warps).  Pick the warp count that wastes the
  // least of the last round.
  int warps = 0;
  long long best = 0;
  {
    const TileSolveLayout l = tile_solve_layout(Bw, T);
    int wmax = (int)((TILE_SMEM_BUDGET - 1024 /* static identity tile */) / l.per_warp_bytes);
    if (wmax > TILE_MAX_WARPS) wmax = TILE_MAX_WARPS;
    for (int w = wmax; w >= 1 && w >= wmax / 2; --w) {
      const long long cost = ceil_div(c, (int64_t)NUM_SMS * w) * w;
      if (warps == 0 || cost < best) {
        best = cost;
        warps = w;
      }
    }
  }
  if (warps < 1) return THANOS_ERR_SHAPE;
  const TileSolveLayout lay = tile_solve_layout(Bw, T);
  const size_t smem = (size_t)warps * lay.per_warp_bytes;
  {
    static std::atomic<unsigned long long> done{0};
    THANOS_CUDA(ensure_max_dyn_smem(solve_rows_tile_kernel, (int)TILE_SMEM_BUDGET - 1024, done));
  }
  int64_t grid = ceil_div(c, warps);
  if (grid > NUM_SMS) grid = NUM_SMS;
  solve_rows_tile_kernel<<<(unsigned)grid, warps * 32, smem, stream>>>(
      Wc, mask, G, S, ld_mat, D, dplane, c, b, j1, Bw, ldd, T, row_lists,
      list_counts, fixed_kind, report_max_s, stats);
  THANOS_CHECK_LAUNCH();
  return THANOS_OK;
}

}  // namespace thanos
