// Per-row constrained solve for large systems (Eqs. 5-8): one CTA per row.
//
// Same mathematics as the warp-per-row kernel (direct form on G for rows with |q| <= |k|,
// complement form on S otherwise), for systems of 97 to 319 unknowns -- e.g. 2:4 sparsity with
// the block width B = 512 of Section 5, where every row solves a 256 x 256 system, or 4:8 with
// B = 256 (128 unknowns).  The gathered
// matrix lives in shared memory as the lower triangle of 16 x 16 tiles (1 KB each, 16-byte chunks
// swizzled by the row so that the accesses below are free of bank conflicts); the right-hand
// side is a vector of its own (as a row of the matrix it would cost a whole extra tile row
// whenever the system size is a multiple of 16, which it always is for n:m masks).
// Right-looking tile Cholesky by the CTA's warps (16, or 4 for the smaller systems; with 16 warps
// the trailing update runs on the tensor cores from bf16 planes of the panel, see below): panel solve (one thread per row), trailing update
// (one warp per target tile, handed out by a shared counter); warp 0 updates and factors the
// next diagonal tile first, which takes the only serial step off the critical path.  Blocked
// substitutions L y = rhs and L^T x = y, then the change of the block's weights as in the small
// kernel.
#include "common.cuh"
#include "tile_ops.cuh"

namespace thanos {

namespace {

using tile::chunk_off;
using tile::elem_off;
using tile::tile_update;

constexpr unsigned FULL = 0xffffffffu;
constexpr int MAX_TILES = 20;  // tile rows: systems of up to 16 * 20 = 320 unknowns (319 are handed out)

// tile (I, J), J <= I, of the lower triangle; 256 floats each
__device__ __forceinline__ int tile_base(int I, int J) { return (((I * (I + 1)) >> 1) + J) << 8; }
__host__ __device__ inline size_t cta_smem_bytes(int tiles, int Bw) {
  // tiles, invd / xs / rhs [16 tiles + 16 each], wblk / dvec [Bw], two index lists, scan scratch
  const size_t fl = (size_t)(tiles * (tiles + 1) / 2) * 256 + 3 * (16 * (size_t)tiles + 16) + 2 * (size_t)Bw;
  return fl * 4 + 2 * 2 * (size_t)(Bw + 16) + 192;
}

// 2 x 2 target tiles (I0 + di, J0 + dj) of step K at once: C_IJ -= L_IK L_JK^T.  Lane (lr, lc)
// owns rows lr, lr + 8 and columns lc + 4 i of every tile, so the operand rows it loads serve
// four tiles.  Bit 2 di + dj of vmask says that the tile is written; tile indices past the last
// tile row are clamped for the loads.
__device__ __forceinline__ void macro_update(float* __restrict__ A, int K, int I0, int J0, int T,
                                             unsigned vmask, int lane) {
  const int lr = lane >> 2, lc = lane & 3;
  const int I1 = I0 + 1 < T ? I0 + 1 : T - 1, J1 = J0 + 1 < T ? J0 + 1 : T - 1;
  const float* At[2] = {A + tile_base(I0, K), A + tile_base(I1, K)};
  const float* Bt[2] = {A + tile_base(J0, K), A + tile_base(J1, K)};
  float acc[2][2][2][4];
#pragma unroll
  for (int di = 0; di < 2; ++di)
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
      for (int dj = 0; dj < 2; ++dj)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[di][h][dj][i] = 0.f;
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    float4 a[2][2], bv[2][4];
#pragma unroll
    for (int di = 0; di < 2; ++di)
#pragma unroll
      for (int h = 0; h < 2; ++h)
        a[di][h] = *reinterpret_cast<const float4*>(At[di] + chunk_off(lr + 8 * h, c));
#pragma unroll
    for (int dj = 0; dj < 2; ++dj)
#pragma unroll
      for (int i = 0; i < 4; ++i)
        bv[dj][i] = *reinterpret_cast<const float4*>(Bt[dj] + chunk_off(lc + 4 * i, c));
#pragma unroll
    for (int di = 0; di < 2; ++di)
#pragma unroll
      for (int dj = 0; dj < 2; ++dj) {
        if (!(vmask & (1u << (2 * di + dj)))) continue;  // warp-uniform
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            float v = acc[di][h][dj][i];
            v = fmaf(a[di][h].x, bv[dj][i].x, v);
            v = fmaf(a[di][h].y, bv[dj][i].y, v);
            v = fmaf(a[di][h].z, bv[dj][i].z, v);
            v = fmaf(a[di][h].w, bv[dj][i].w, v);
            acc[di][h][dj][i] = v;
          }
      }
  }
#pragma unroll
  for (int di = 0; di < 2; ++di)
#pragma unroll
    for (int dj = 0; dj < 2; ++dj) {
      if (!(vmask & (1u << (2 * di + dj)))) continue;
      float* Ct = A + tile_base(I0 + di, J0 + dj);
#pragma unroll
      for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int i = 0; i < 4; ++i) Ct[chunk_off(lr + 8 * h, i) + lc] -= acc[di][h][dj][i];
    }
}

// ---- trailing update on the tensor cores: the rows of the current panel are kept a second time
// as three bf16 planes (x = h + m + l, 24 significant bits; row stride 24 elements, which makes
// the fragment loads below free of bank conflicts), and C_IJ -= L_IK L_JK^T is the sum of the six
// plane products hh, hm, mh, hl, lh, mm by mma.sync m16n8k16 with fp32 accumulation.
constexpr int PLANE_LD = 24;

__device__ __forceinline__ void mma_bf16_m16n8k16(float (&d)[4], const uint32_t (&a)[4],
                                                  const uint32_t (&b)[2]) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

// planes of one solved panel row (16 values read back from its tile)
__device__ __forceinline__ void store_row_planes(const float* __restrict__ tile_row_src, int r,
                                                 __nv_bfloat16* __restrict__ prow, int plane_stride) {
  float x[16];
#pragma unroll
  for (int cc = 0; cc < 4; ++cc) {
    const float4 v = *reinterpret_cast<const float4*>(tile_row_src + tile::chunk_off(r, cc));
    x[4 * cc] = v.x; x[4 * cc + 1] = v.y; x[4 * cc + 2] = v.z; x[4 * cc + 3] = v.w;
  }
#pragma unroll
  for (int pl = 0; pl < 3; ++pl) {
    uint32_t w[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      // two values per conversion; the low half of the word is the lower column
      const __nv_bfloat162 pr = __floats2bfloat162_rn(x[2 * e], x[2 * e + 1]);
      w[e] = *reinterpret_cast<const uint32_t*>(&pr);
      if (pl < 2) {
        x[2 * e] -= __uint_as_float(w[e] << 16);
        x[2 * e + 1] -= __uint_as_float(w[e] & 0xffff0000u);
      }
    }
    uint4* dst = reinterpret_cast<uint4*>(prow + (size_t)pl * plane_stride);
    dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
    dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
  }
}

// 2 x 2 target tiles (I0 + di, J0 + dj) of step K from the panel's planes.  pa / pb: first panel
// row of the tiles I0 / J0.  Fragment layout of mma.m16n8k16 (g = lane / 4, t = lane % 4):
// A: rows g, g + 8, columns 2t, 2t + 1 (+8);  B: column g of the 8, rows (= k) 2t, 2t + 1 (+8);
// C: rows g, g + 8, columns 2t, 2t + 1 of the 8.
__device__ __forceinline__ void macro_update_mma(float* __restrict__ A, int K, int I0, int J0, int T,
                                                 unsigned vmask, const __nv_bfloat16* __restrict__ Pp,
                                                 int plane_stride, int lane) {
  const int g = lane >> 2, t = lane & 3;
  const int m = T - K - 1;  // tile rows in the panel
  uint32_t af[2][3][4], bf[2][3][2][2];
#pragma unroll
  for (int d = 0; d < 2; ++d) {
    const int ti = min(I0 - K - 1 + d, m - 1), tj = min(J0 - K - 1 + d, m - 1);  // clamped loads
#pragma unroll
    for (int pl = 0; pl < 3; ++pl) {
      const __nv_bfloat16* pa = Pp + (size_t)pl * plane_stride + (size_t)(16 * ti) * PLANE_LD;
      const __nv_bfloat16* pb = Pp + (size_t)pl * plane_stride + (size_t)(16 * tj) * PLANE_LD;
      af[d][pl][0] = *reinterpret_cast<const uint32_t*>(pa + g * PLANE_LD + 2 * t);
      af[d][pl][1] = *reinterpret_cast<const uint32_t*>(pa + (g + 8) * PLANE_LD + 2 * t);
      af[d][pl][2] = *reinterpret_cast<const uint32_t*>(pa + g * PLANE_LD + 2 * t + 8);
      af[d][pl][3] = *reinterpret_cast<const uint32_t*>(pa + (g + 8) * PLANE_LD + 2 * t + 8);
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        bf[d][pl][h][0] = *reinterpret_cast<const uint32_t*>(pb + (8 * h + g) * PLANE_LD + 2 * t);
        bf[d][pl][h][1] = *reinterpret_cast<const uint32_t*>(pb + (8 * h + g) * PLANE_LD + 2 * t + 8);
      }
    }
  }
#pragma unroll
  for (int di = 0; di < 2; ++di)
#pragma unroll
    for (int dj = 0; dj < 2; ++dj) {
      if (!(vmask & (1u << (2 * di + dj)))) continue;  // warp-uniform
      float* Ct = A + tile_base(I0 + di, J0 + dj);
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        // smallest products first
        mma_bf16_m16n8k16(acc, af[di][1], bf[dj][1][h]);  // m m
        mma_bf16_m16n8k16(acc, af[di][2], bf[dj][0][h]);  // l h
        mma_bf16_m16n8k16(acc, af[di][0], bf[dj][2][h]);  // h l
        mma_bf16_m16n8k16(acc, af[di][1], bf[dj][0][h]);  // m h
        mma_bf16_m16n8k16(acc, af[di][0], bf[dj][1][h]);  // h m
        mma_bf16_m16n8k16(acc, af[di][0], bf[dj][0][h]);  // h h
        float2* c0 = reinterpret_cast<float2*>(Ct + tile::elem_off(g, 8 * h + 2 * t));
        float2* c1 = reinterpret_cast<float2*>(Ct + tile::elem_off(g + 8, 8 * h + 2 * t));
        float2 v0 = *c0, v1 = *c1;
        v0.x -= acc[0]; v0.y -= acc[1];
        v1.x -= acc[2]; v1.y -= acc[3];
        *c0 = v0;
        *c1 = v1;
      }
    }
}

// The same 2 x 2 group without stored planes: the fp32 panel tiles are split into bf16 planes in
// registers (tile_ops.cuh), so a group costs four fragment loads, 48 tensor-core instructions and
// the read-modify-write of its targets.  For the four-warp CTAs, whose shared memory has no room
// for the planes of a panel.
__device__ __forceinline__ void macro_update_frag(float* __restrict__ A, int K, int I0, int J0, int T,
                                                  unsigned vmask, const tile::FragOff& fo) {
  const int I1 = I0 + 1 < T ? I0 + 1 : T - 1, J1 = J0 + 1 < T ? J0 + 1 : T - 1;
  tile::PanelFrag fa[2], fb[2];
  tile::load_panel_frag(A + tile_base(I0, K), fo, fa[0]);
  tile::load_panel_frag(A + tile_base(I1, K), fo, fa[1]);
  tile::load_panel_frag(A + tile_base(J0, K), fo, fb[0]);
  tile::load_panel_frag(A + tile_base(J1, K), fo, fb[1]);
#pragma unroll
  for (int di = 0; di < 2; ++di)
#pragma unroll
    for (int dj = 0; dj < 2; ++dj) {
      if (!(vmask & (1u << (2 * di + dj)))) continue;  // warp-uniform
      float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
      tile::frag_product(acc, fa[di], fb[dj]);
      tile::tile_subtract(A + tile_base(I0 + di, J0 + dj), acc, fo);
    }
}

// exclusive prefix sum of one value per thread over the CTA
template <int CTA_WARPS>
__device__ __forceinline__ unsigned cta_exclusive_scan(unsigned x, unsigned* warp_sums,
                                                       unsigned& total) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  unsigned incl = x;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned y = __shfl_up_sync(FULL, incl, o);
    if (lane >= o) incl += y;
  }
  __syncthreads();
  if (lane == 31) warp_sums[wid] = incl;
  __syncthreads();
  unsigned before = 0, all = 0;
#pragma unroll
  for (int w = 0; w < CTA_WARPS; ++w) {
    const unsigned v = warp_sums[w];
    if (w < wid) before += v;
    all += v;
  }
  total = all;
  return before + incl - x;
}

// Rows come from row_lists[2][c] / list_counts[2] (kind 0: |q| <= |k|, direct form on G; kind 1:
// complement form on S), or are all rows with kind `fixed_kind` when row_lists is null.
//
// CTA_THREADS = 512: one CTA per SM, for the largest systems (the tiles of one row fill most of the
// shared memory).  CTA_THREADS = 128: four CTAs per SM for systems of 96 to 159 unknowns, where
// four rows in flight with four warps each beat both one row with sixteen warps and the
// warp-per-row kernel (whose 41 KB per warp leave room for five rows per SM).
template <int CTA_THREADS>
__global__ void __launch_bounds__(CTA_THREADS, CTA_THREADS == 128 ? 5 : 512 / CTA_THREADS)
solve_rows_cta_kernel(float* __restrict__ Wc, const uint8_t* __restrict__ mask,
                      const float* __restrict__ Gm, const float* __restrict__ Sm, int ld_mat,
                      __nv_bfloat16* __restrict__ D, int64_t dplane, int c, int b, int j1, int Bw,
                      int ldd, int tiles, const int* __restrict__ row_lists,
                      const unsigned* __restrict__ list_counts, int fixed_kind, int report_max_s,
                      int use_planes, thanos_stats_t* stats) {
  extern __shared__ __align__(16) unsigned char dyn[];
  const int tid = threadIdx.x;
  const int lane = tid & 31;
  const int warp = tid >> 5;
  float* A = reinterpret_cast<float*>(dyn);
  float* invd = A + (size_t)(tiles * (tiles + 1) / 2) * 256;
  float* xs = invd + 16 * tiles + 16;
  float* rhsv = xs + 16 * tiles + 16;
  float* wblk = rhsv + 16 * tiles + 16;
  float* dvec = wblk + Bw;
  unsigned short* qlist = reinterpret_cast<unsigned short*>(dvec + Bw);
  unsigned short* klist = qlist + Bw + 16;
  unsigned* scratch = reinterpret_cast<unsigned*>(klist + Bw + 16);  // 48 words
  unsigned* warp_sums = scratch;          // [32]
  unsigned* s_counter = scratch + 32;
  unsigned* s_bad = scratch + 33;
  // planes of the current panel (tensor-core trailing update), 16-byte aligned behind the scratch
  __nv_bfloat16* Pp = reinterpret_cast<__nv_bfloat16*>(
      dyn + ((reinterpret_cast<unsigned char*>(scratch + 48) - dyn + 15) & ~(size_t)15));
  const int plane_stride = 16 * (tiles - 1) * PLANE_LD;
  const tile::FragOff frag_off = tile::make_frag_off(lane >> 2, lane & 3);

  int cnt0, cnt1;
  if (row_lists) {
    cnt0 = (int)list_counts[0];
    cnt1 = (int)list_counts[1];
  } else {
    cnt0 = fixed_kind == 0 ? c : 0;
    cnt1 = fixed_kind == 0 ? 0 : c;
  }
  for (int li = blockIdx.x; li < cnt0 + cnt1; li += gridDim.x) {
    const bool kpath = li >= cnt0;
    const int row = row_lists ? (kpath ? row_lists[(size_t)c + (li - cnt0)] : row_lists[li]) : li;
    const float* __restrict__ M = kpath ? Sm : Gm;
    const uint8_t* mrow = mask + (int64_t)row * b + j1;
    float* wrow = Wc + (int64_t)row * b + j1;
    __syncthreads();  // the previous row's shared data is no longer read
    // ---- q = phi(mask row) and its complement k, both ascending: thread t owns columns 2t, 2t+1
    int s, t;
    {
      const int c0 = 2 * tid, c1 = 2 * tid + 1;
      const int m0 = c0 < Bw ? (int)mrow[c0] : 2, m1 = c1 < Bw ? (int)mrow[c1] : 2;
      if (c0 < Bw) wblk[c0] = wrow[c0];
      if (c1 < Bw) wblk[c1] = wrow[c1];
      const unsigned mine = (unsigned)((m0 == 1) + (m1 == 1)) | ((unsigned)((m0 == 0) + (m1 == 0)) << 16);
      unsigned all;
      const unsigned before = cta_exclusive_scan<CTA_THREADS / 32>(mine, warp_sums, all);
      int pq = (int)(before & 0xffffu), pk = (int)(before >> 16);
      if (m0 == 1) qlist[pq++] = (unsigned short)c0;
      if (m0 == 0) klist[pk++] = (unsigned short)c0;
      if (m1 == 1) qlist[pq] = (unsigned short)c1;
      if (m1 == 0) klist[pk] = (unsigned short)c1;
      s = (int)(all & 0xffffu);
      t = (int)(all >> 16);
    }
    if (tid == 0) *s_bad = 0;
    if (s == 0) {  // nothing removed: the row is not touched in this block (CTA-uniform)
      for (int jj = tid; jj < Bw; jj += CTA_THREADS) store_split3(D + (int64_t)row * ldd + jj, dplane, 0.f);
      continue;
    }
    if (report_max_s && row == 0 && tid == 0) atomicMax(&stats->max_s, s);
    const int n = kpath ? t : s;   // unknowns of this row's system
    const int no = kpath ? s : t;  // size of the other set
    unsigned short* sel = kpath ? klist : qlist;
    unsigned short* oth = kpath ? qlist : klist;
    if (tid < 16) {
      sel[n + tid] = 0;
      oth[no + tid] = 0;
    }
    const int T = (n + 15) >> 4;   // tile rows (= tile columns) of the system
    const int Tf = T;
    if ((s > t) != kpath || T > tiles) {
      // cannot happen for lists and launch sizes made by this library
      if (tid == 0) report_error(&stats->status, THANOS_ERR_SHAPE, row);
      for (int jj = tid; jj < Bw; jj += CTA_THREADS) store_split3(D + (int64_t)row * ldd + jj, dplane, 0.f);
      continue;
    }
    __syncthreads();
    // ---- right-hand side: w_q (direct form) or g_e = sum_a w[q_a] S[q_a, k_e] (complement)
    for (int e = tid; e < n; e += CTA_THREADS) {
      float g;
      if (!kpath) {
        g = wblk[sel[e]];
      } else {
        const int col = (int)sel[e];
        float g0 = 0.f, g1 = 0.f;
        for (int a = 0; a < no; a += 4) {
          const ushort4 ix = *reinterpret_cast<const ushort4*>(oth + a);
          const float w0 = wblk[ix.x];
          const float w1 = (a + 1 < no) ? wblk[ix.y] : 0.f;
          const float w2 = (a + 2 < no) ? wblk[ix.z] : 0.f;
          const float w3 = (a + 3 < no) ? wblk[ix.w] : 0.f;
          g0 = fmaf(w0, __ldg(M + (int)ix.x * ld_mat + col), g0);
          g1 = fmaf(w1, __ldg(M + (int)ix.y * ld_mat + col), g1);
          g0 = fmaf(w2, __ldg(M + (int)ix.z * ld_mat + col), g0);
          g1 = fmaf(w3, __ldg(M + (int)ix.w * ld_mat + col), g1);
        }
        g = g0 + g1;
      }
      rhsv[e] = g;
    }
    __syncthreads();
    // ---- gather the lower triangle of M[sel, sel], identity padding
    {
      // A tile has 256 entries: with 512 threads two tiles are filled at a time, with 128 threads
      // a thread fills two entries of each tile; eight tiles' loads are in flight per thread.
      constexpr int GROUPS = CTA_THREADS >= 256 ? CTA_THREADS / 256 : 1;  // tiles at a time
      constexpr int PER = CTA_THREADS >= 256 ? 1 : 256 / CTA_THREADS;     // entries per thread and tile
      constexpr int RSTEP = CTA_THREADS >= 256 ? 16 : CTA_THREADS / 16;   // row step between them
      const int r0 = (tid & 255) >> 4, k = tid & 15, grp = tid >> 8;
      const int ntiles = (T * (T + 1)) >> 1;
      int I = 0, J = 0;
      for (int g = 0; g < grp; ++g)
        if (++J > I) {
          ++I;
          J = 0;
        }
      for (int t0 = grp; t0 < ntiles; t0 += 8 * GROUPS) {
        float v[8][PER];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
#pragma unroll
          for (int h = 0; h < PER; ++h) {
            const int r = r0 + RSTEP * h;
            const int i = 16 * I + r, j = 16 * J + k;
            float x;
            if (t0 + u * GROUPS >= ntiles)
              x = 0.f;
            else if (i < n)
              x = j < n ? __ldg(M + (int)sel[i] * ld_mat + (int)sel[j]) : 0.f;
            else
              x = i == j ? 1.f : 0.f;
            v[u][h] = x;
          }
#pragma unroll
          for (int g = 0; g < GROUPS; ++g)
            if (++J > I) {
              ++I;
              J = 0;
            }
        }
#pragma unroll
        for (int u = 0; u < 8; ++u)
#pragma unroll
          for (int h = 0; h < PER; ++h)
            if (t0 + u * GROUPS < ntiles)
              A[((t0 + u * GROUPS) << 8) + elem_off(r0 + RSTEP * h, k)] = v[u][h];
      }
    }
    __syncthreads();
    bool bad = false;
    if (warp == 0 && T > 0) bad = tile::factor_diag_tile<false>(A + tile_base(0, 0), invd, 0, n, lane) >= 0;
    for (int i = tid; i < 16 * T + 4; i += CTA_THREADS) xs[i] = i < n ? rhsv[i] : 0.f;
    __syncthreads();
    // ---- right-looking tile Cholesky; the forward substitution L y = rhs rides along: tile
    //      column K of y is solved by the last warp at the start of step K (L_KK is factored and
    //      xs[16 K ..] has received every earlier column by then), and the entries below it are
    //      updated with the solved panel at the start of the trailing phase
    for (int K = 0; K < Tf; ++K) {
      const int m = T - K - 1;  // tile rows below the diagonal tile
      if (tid == 0) *s_counter = 0;
      if (warp == CTA_THREADS / 32 - 1) {
        const float* Lk = A + tile_base(K, K);
        const int me = 16 * K + (lane & 15);
        float res = me < n ? xs[me] : 0.f;
#pragma unroll
        for (int w = 0; w < 16; ++w) {
          const int idx = 16 * K + w;
          float yi = __shfl_sync(FULL, res, w);
          yi = idx < n ? yi * invd[idx] : 0.f;
          const float lkw = Lk[elem_off(lane & 15, w)];
          if ((lane & 15) > w) res = fmaf(-lkw, yi, res);
          if ((lane & 15) == w) res = yi;
        }
        if (lane < 16 && me < n) xs[me] = res;
      }
      // panel: X L_KK^T = A_IK for the rows below, one thread per row
      {
        const float* Lk = A + tile_base(K, K);
        for (int ii = tid; ii < 16 * m; ii += CTA_THREADS) {
          const int I = K + 1 + (ii >> 4), r = ii & 15;
          tile::panel_row_solve(A + tile_base(I, K), r, Lk, invd + 16 * K);
          if (use_planes) store_row_planes(A + tile_base(I, K), r, Pp + (size_t)ii * PLANE_LD, plane_stride);
        }
      }
      __syncthreads();
      // right-hand side below tile row K: xs[k] -= L[k, 16 K ..] y_K
      for (int k = 16 * (K + 1) + tid; k < 16 * T; k += CTA_THREADS) {
        const float* Lt = A + tile_base(k >> 4, K);
        const int kk = k & 15;
        float acc = 0.f;
#pragma unroll
        for (int w = 0; w < 16; ++w) acc = fmaf(Lt[elem_off(kk, w)], xs[16 * K + w], acc);
        xs[k] -= acc;
      }
      // trailing update; warp 0 first brings the next diagonal tile up to date and factors it
      if (warp == 0 && K + 1 < Tf) {
        float* Ct = A + tile_base(K + 1, K + 1);
        const float* At = A + tile_base(K + 1, K);
        tile_update(Ct, At, At, lane);
        __syncwarp();
        bad |= tile::factor_diag_tile<false>(Ct, invd, 16 * (K + 1), n, lane) >= 0;
      }
      {
        // the m x m lower triangle of targets in 2 x 2 groups (I', J') in row-major order,
        // handed out by the shared counter; the next diagonal tile (done by warp 0 above) and a
        // last column that is not factored are masked out
        const int m2 = (m + 1) >> 1;
        const int total = (m2 * (m2 + 1)) >> 1;
        for (;;) {
          unsigned u = 0;
          if (lane == 0) u = atomicAdd(s_counter, 1u);
          u = __shfl_sync(FULL, u, 0);
          if ((int)u >= total) break;
          int Ip = (int)((sqrtf(8.f * (float)u + 1.f) - 1.f) * 0.5f);
          while (((Ip + 1) * (Ip + 2) >> 1) <= (int)u) ++Ip;
          while (((Ip * (Ip + 1)) >> 1) > (int)u) --Ip;
          const int Jp = (int)u - ((Ip * (Ip + 1)) >> 1);
          const int I0 = K + 1 + 2 * Ip, J0 = K + 1 + 2 * Jp;
          unsigned vmask = 0;
#pragma unroll
          for (int di = 0; di < 2; ++di)
#pragma unroll
            for (int dj = 0; dj < 2; ++dj) {
              const int I = I0 + di, J = J0 + dj;
              if (I < T && J <= I && J < Tf && !(I == K + 1 && J == K + 1)) vmask |= 1u << (2 * di + dj);
            }
          if (vmask) {
            if (use_planes)
              macro_update_mma(A, K, I0, J0, T, vmask, Pp, plane_stride, lane);
            else if (CTA_THREADS == 128)
              macro_update_frag(A, K, I0, J0, T, vmask, frag_off);
            else
              macro_update(A, K, I0, J0, T, vmask, lane);
          }
        }
      }
      __syncthreads();
    }
    if (warp == 0 && bad && lane == 0) *s_bad = 1;
    __syncthreads();
    if (*s_bad) {
      if (tid == 0) report_error(&stats->status, THANOS_ERR_NOT_SPD, row);
      for (int jj = tid; jj < Bw; jj += CTA_THREADS) store_split3(D + (int64_t)row * ldd + jj, dplane, 0.f);
      continue;
    }
    // ---- blocked back substitution L^T x = y from the bottom
    for (int Kb = Tf - 1; Kb >= 0; --Kb) {
      if (warp == 0) {
        const float* Lk = A + tile_base(Kb, Kb);
        const int me = 16 * Kb + (lane & 15);
        float res = me < n ? xs[me] : 0.f;
#pragma unroll
        for (int w = 15; w >= 0; --w) {
          const int idx = 16 * Kb + w;
          float xi = __shfl_sync(FULL, res, w);
          xi = idx < n ? xi * invd[idx] : 0.f;
          const float lwk = Lk[elem_off(w, lane & 15)];
          if ((lane & 15) < w) res = fmaf(-lwk, xi, res);
          if ((lane & 15) == w) res = xi;
        }
        if (lane < 16 && me < n) xs[me] = res;
      }
      __syncthreads();
      for (int k = tid; k < 16 * Kb; k += CTA_THREADS) {
        const float* Lt = A + tile_base(Kb, k >> 4);
        const int kk = k & 15;
        float acc = 0.f;
#pragma unroll
        for (int w = 0; w < 16; ++w) acc = fmaf(Lt[elem_off(w, kk)], xs[16 * Kb + w], acc);
        xs[k] -= acc;
      }
      __syncthreads();
    }
    // ---- delta over the block
    for (int a = tid; a < s; a += CTA_THREADS) dvec[qlist[a]] = -wblk[qlist[a]];
    __syncthreads();
    if (kpath) {
      for (int e = tid; e < n; e += CTA_THREADS) dvec[sel[e]] = xs[e];
    } else {
      // delta_k = -sum_a lambda_a G[q_a, k_e]
      for (int e = tid; e < no; e += CTA_THREADS) {
        const int col = (int)oth[e];
        float g0 = 0.f, g1 = 0.f, g2 = 0.f, g3 = 0.f;
        for (int a = 0; a < n; a += 4) {
          const ushort4 ix = *reinterpret_cast<const ushort4*>(sel + a);
          const float4 xv = *reinterpret_cast<const float4*>(xs + a);
          g0 = fmaf(xv.x, __ldg(M + (int)ix.x * ld_mat + col), g0);
          g1 = fmaf(xv.y, __ldg(M + (int)ix.y * ld_mat + col), g1);
          g2 = fmaf(xv.z, __ldg(M + (int)ix.z * ld_mat + col), g2);
          g3 = fmaf(xv.w, __ldg(M + (int)ix.w * ld_mat + col), g3);
        }
        dvec[col] = -((g0 + g1) + (g2 + g3));
      }
    }
    __syncthreads();
    for (int jj = tid; jj < Bw; jj += CTA_THREADS) {
      const float d = dvec[jj];
      const bool removed = mrow[jj] != 0;
      wrow[jj] = removed ? 0.f : wblk[jj] + d;
      store_split3(D + (int64_t)row * ldd + jj, dplane, d);
    }
  }
}

}  // namespace

// Largest system (unknowns) the CTA-per-row kernel holds.
int cta_solve_max_unknowns() { return 16 * MAX_TILES - 1; }

template <int CTA_THREADS>
thanos_status_t launch_cta_solve_t(float* Wc, const uint8_t* mask, const float* G, const float* S,
                                   int ld_mat, __nv_bfloat16* D, int64_t dplane, int c, int b,
                                   int j1, int Bw, int ldd, int tiles, size_t smem, int use_planes,
                                   const int* row_lists, const unsigned* list_counts,
                                   int fixed_kind, int report_max_s, thanos_stats_t* stats,
                                   cudaStream_t stream) {
  {
    static std::atomic<unsigned long long> done{0};
    THANOS_CUDA(ensure_max_dyn_smem(solve_rows_cta_kernel<CTA_THREADS>, 227 * 1024, done));
  }
  // CTAs per SM: what the shared memory of a CTA (plus the 1 KB the system keeps per CTA) allows,
  // up to five of the four-warp CTAs
  int per_sm = 512 / CTA_THREADS;
  if (CTA_THREADS == 128) {
    per_sm = (int)((228 * 1024) / (smem + 1024));
    per_sm = per_sm < 1 ? 1 : (per_sm > 5 ? 5 : per_sm);
  }
  const int ctas = NUM_SMS * per_sm;
  const int grid = c < ctas ? c : ctas;
  solve_rows_cta_kernel<CTA_THREADS><<<(unsigned)grid, CTA_THREADS, smem, stream>>>(
      Wc, mask, G, S, ld_mat, D, dplane, c, b, j1, Bw, ldd, tiles, row_lists, list_counts,
      fixed_kind, report_max_s, use_planes, stats);
  THANOS_CHECK_LAUNCH();
  return THANOS_OK;
}

thanos_status_t launch_cta_solve(float* Wc, const uint8_t* mask, const float* G, const float* S,
                                 int ld_mat, __nv_bfloat16* D, int64_t dplane, int c, int b, int j1,
                                 int Bw, int ldd, int n_max, const int* row_lists,
                                 const unsigned* list_counts, int fixed_kind, int report_max_s,
                                 thanos_stats_t* stats, cudaStream_t stream) {
  const int tiles = (n_max + 15) / 16 > 0 ? (n_max + 15) / 16 : 1;
  if (tiles > MAX_TILES || Bw > 1024) return THANOS_ERR_SHAPE;
  const size_t smem = cta_smem_bytes(tiles, Bw);
  if (smem > 227 * 1024) return THANOS_ERR_SHAPE;
  // small tile sets: four CTAs of four warps per SM (a thread owns two columns of the block)
  if (smem <= 56 * 1024 && Bw <= 256)
    return launch_cta_solve_t<128>(Wc, mask, G, S, ld_mat, D, dplane, c, b, j1, Bw, ldd, tiles, smem, 0,
                                   row_lists, list_counts, fixed_kind, report_max_s, stats, stream);
  // the planes of a panel (tensor-core trailing update) when they still fit next to the tiles
  const size_t with_planes = ((smem + 15) & ~(size_t)15) + 3 * (size_t)16 * (tiles - 1) * PLANE_LD * 2;
  const int use_planes = with_planes <= 227 * 1024 ? 1 : 0;
  return launch_cta_solve_t<512>(Wc, mask, G, S, ld_mat, D, dplane, c, b, j1, Bw, ldd, tiles,
                                 use_planes ? with_planes : smem, use_planes,
                                 row_lists, list_counts, fixed_kind, report_max_s, stats, stream);
}

}  // namespace thanos
