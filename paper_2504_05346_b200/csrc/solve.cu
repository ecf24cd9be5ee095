// Per-row constrained solve of one block step (Eqs. 5-8): for every row, with q = phi(mask row)
// the removed positions inside the block and k the kept ones, the optimal change of the block's
// weights.
//
// Notation: G = inv(H_d[j1:, j1:])[0:B, 0:B] (the block of the residual inverse) and
// S = inv(G) (the Schur complement of the residual Hessian onto the block).  Eq. 8 restricted to
// the block reads  delta_k = -lambda-hat G[q, k]  with  lambda-hat G[q, q] = w_q  (Eqs. 6-7); the
// same minimiser is  delta_k S[k, k] = w_q S[q, k]  (stationarity of delta S delta^T in the free
// coordinates), which is the smaller system whenever more than half of the block is removed.
// Each row therefore solves a system of min(|q|, |k|) unknowns:
//   direct form      lambda-hat = G[q,q]^{-1} w_q,   delta_k = -lambda-hat G[q, k]
//   complement form  delta_k = S[k,k]^{-1} (S[k,q] w_q)
// and in both forms delta_q = -w_q.  The rows of a block are independent.
//
// Fast kernel: one warp per row.  The gathered matrix lives in shared memory as a packed lower
// triangle whose rows are padded so that eight consecutive rows never share a bank group; the
// right-hand side is appended as one more row, so the factorisation L L^T also yields
// L^{-1} rhs.  Left-looking Cholesky in panels of 8 columns: a lane owns up to NR rows of the
// panel (8 accumulators each), the 8 x 8 diagonal block is factored with warp shuffles.
// Systems of 160 unknowns and more go to the CTA-per-row kernel of solve_cta.cu.
#include "common.cuh"

namespace thanos {

namespace {

constexpr unsigned FULL = 0xffffffffu;

__host__ __device__ __forceinline__ int tri_row_off(int r) {
  // rows 8m .. 8m+7 have 8m + 12 floats each (8m + 8 columns plus a 4-float skew)
  const int m = r >> 3, t = r & 7;
  return 32 * m * m + 64 * m + t * (8 * m + 12);
}
__host__ __device__ __forceinline__ int tri_floats(int panels) {
  return 32 * panels * panels + 64 * panels;
}

struct SolveSmemLayout {
  int mat_floats;      // shared copy of G or S (0 when it stays in global memory)
  int ldm;             // its leading dimension
  int per_warp_bytes;  // one warp's scratch
  int a_floats, vec_floats, list_elems;
};

__host__ __device__ inline SolveSmemLayout solve_layout(int Bw, int panels, bool mat_in_smem) {
  SolveSmemLayout L;
  L.ldm = mat_in_smem ? (Bw | 1) : 0;
  L.mat_floats = mat_in_smem ? ((Bw * L.ldm + 3) & ~3) : 0;
  L.a_floats = tri_floats(panels);
  L.vec_floats = Bw;
  L.list_elems = Bw + 16;
  // A, invd[8 panels], rhs[8 panels + 8], wblk[Bw], dvec[Bw], two index lists
  int bytes = 4 * (L.a_floats + 16 * panels + 8 + 2 * L.vec_floats) + 2 * 2 * L.list_elems;
  L.per_warp_bytes = (bytes + 15) & ~15;
  return L;
}

// One warp per row.  A CTA serves one kind of row: kind 0 = rows with |q| <= |k| (direct form,
// matrix G), kind 1 = rows with |q| > |k| (complement form, matrix S); its matrix sits in shared
// memory.  With row lists (unstructured mode: the mask kernel sorts the rows by kind) the CTAs
// are split between the kinds in proportion to the list lengths; without them every row is of
// kind `fixed_kind`.
template <int NR>
__global__ void __launch_bounds__(32 * 15)
solve_rows_fast_kernel(float* __restrict__ Wc, const uint8_t* __restrict__ mask,
                       const float* __restrict__ Gm, const float* __restrict__ Sm, int ld_mat,
                       __nv_bfloat16* __restrict__ D, int64_t dplane, int c, int b, int j1, int Bw, int ldd,
                       int panels,
                       int mat_in_smem, const int* __restrict__ row_lists,
                       const unsigned* __restrict__ list_counts, int fixed_kind, int report_max_s,
                       thanos_stats_t* stats) {
  extern __shared__ __align__(16) unsigned char dyn[];
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int warps = blockDim.x >> 5;
  const SolveSmemLayout lay = solve_layout(Bw, panels, mat_in_smem != 0);
  float* Ms = reinterpret_cast<float*>(dyn);
  unsigned char* wbase = dyn + 4 * (size_t)lay.mat_floats + (size_t)warp * lay.per_warp_bytes;
  float* A = reinterpret_cast<float*>(wbase);
  float* invd = A + lay.a_floats;
  float* rhsv = invd + 8 * panels;
  float* wblk = rhsv + 8 * panels + 8;
  float* dvec = wblk + lay.vec_floats;
  unsigned short* qlist = reinterpret_cast<unsigned short*>(dvec + lay.vec_floats);
  unsigned short* klist = qlist + lay.list_elems;

  int cnt[2];
  if (row_lists) {
    cnt[0] = (int)list_counts[0];
    cnt[1] = (int)list_counts[1];
  } else {
    cnt[fixed_kind] = c;
    cnt[fixed_kind ^ 1] = 0;
  }
  const int nctas = gridDim.x;
  // CTAs [0, nctas - n1) serve kind 0, the rest kind 1
  int n1 = 0;
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
    const float* Mat = kpath ? Sm : Gm;
    const float* M;
    int ldm;
    if (mat_in_smem) {
      __syncthreads();
      const int q4 = Bw >> 2;
      for (int i = warp; i < Bw; i += warps) {
        const float4* src = reinterpret_cast<const float4*>(Mat + (int64_t)i * ld_mat);
        for (int j = lane; j < q4; j += 32) {
          const float4 v = src[j];
          float* dst = Ms + i * lay.ldm + 4 * j;
          dst[0] = v.x; dst[1] = v.y; dst[2] = v.z; dst[3] = v.w;
        }
      }
      __syncthreads();
      M = Ms;
      ldm = lay.ldm;
    } else {
      M = Mat;
      ldm = ld_mat;
    }
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
      const int n_pad = (n + 1 + 7) & ~7;  // the system, the right-hand-side row, identity padding
      if ((s > t) != kpath || n_pad > 8 * panels || n_pad > 32 * NR) {
        // cannot happen for lists and launch sizes made by this library
        if (lane == 0) report_error(&stats->status, THANOS_ERR_SHAPE, row);
        __syncwarp();
        continue;
      }
      __syncwarp();
      // ---- right-hand side: w_q (direct form) or g_e = sum_a w[q_a] S[q_a, k_e] (complement)
      for (int e0 = 0; e0 < n_pad + 8; e0 += 32) {
        const int e = e0 + lane;
        float g = 0.f;
        if (!kpath) {
          if (e < n) g = wblk[sel[e]];
        } else {
          const int col = (e < n) ? (int)sel[e] : 0;
          for (int a = 0; a < no; a += 4) {
            const ushort4 ix = *reinterpret_cast<const ushort4*>(oth + a);
            const float w0 = wblk[ix.x];
            const float w1 = (a + 1 < no) ? wblk[ix.y] : 0.f;
            const float w2 = (a + 2 < no) ? wblk[ix.z] : 0.f;
            const float w3 = (a + 3 < no) ? wblk[ix.w] : 0.f;
            g = fmaf(w0, M[(int)ix.x * ldm + col], g);
            g = fmaf(w1, M[(int)ix.y * ldm + col], g);
            g = fmaf(w2, M[(int)ix.z * ldm + col], g);
            g = fmaf(w3, M[(int)ix.w * ldm + col], g);
          }
          if (e >= n) g = 0.f;
        }
        if (e == n) g = 1.f;  // diagonal of the appended row (its pivot is never used)
        if (e < n_pad + 8) rhsv[e] = g;
      }
      __syncwarp();

      // ---- left-looking Cholesky, panels of 8 columns; entries are gathered as they are needed
      bool bad = false;
      for (int c0 = 0; c0 < n_pad; c0 += 8) {
        float acc[NR][8];
        int off[NR];
        bool valid[NR];
        const int rows_left = n_pad - c0;
        const ushort4 cl = *reinterpret_cast<const ushort4*>(sel + c0);
        const ushort4 ch = *reinterpret_cast<const ushort4*>(sel + c0 + 4);
        const float4 rl = *reinterpret_cast<const float4*>(rhsv + c0);
        const float4 rh = *reinterpret_cast<const float4*>(rhsv + c0 + 4);
#pragma unroll
        for (int r = 0; r < NR; ++r) {
          const int i = c0 + lane + 32 * r;
          valid[r] = i < n_pad;
          off[r] = tri_row_off(valid[r] ? i : c0);
          if (32 * r < rows_left) {
            if (i < n) {
              const float* Mrow = M + (int)sel[i] * ldm;
              acc[r][0] = Mrow[cl.x]; acc[r][1] = Mrow[cl.y];
              acc[r][2] = Mrow[cl.z]; acc[r][3] = Mrow[cl.w];
              acc[r][4] = Mrow[ch.x]; acc[r][5] = Mrow[ch.y];
              acc[r][6] = Mrow[ch.z]; acc[r][7] = Mrow[ch.w];
            } else if (i == n) {
              acc[r][0] = rl.x; acc[r][1] = rl.y; acc[r][2] = rl.z; acc[r][3] = rl.w;
              acc[r][4] = rh.x; acc[r][5] = rh.y; acc[r][6] = rh.z; acc[r][7] = rh.w;
            } else {
#pragma unroll
              for (int w = 0; w < 8; ++w) acc[r][w] = (c0 + w == i) ? 1.f : 0.f;
            }
          } else {
#pragma unroll
            for (int w = 0; w < 8; ++w) acc[r][w] = 0.f;
          }
        }
        const float* Pb = A + tri_row_off(c0);
        const int pstride = c0 + 12;  // row length inside the panel's group of 8 rows
        for (int k = 0; k < c0; k += 4) {
          float4 bv[8];
#pragma unroll
          for (int w = 0; w < 8; ++w) bv[w] = *reinterpret_cast<const float4*>(Pb + w * pstride + k);
#pragma unroll
          for (int r = 0; r < NR; ++r) {
            if (32 * r < rows_left) {  // warp-uniform
              const float4 av = *reinterpret_cast<const float4*>(A + off[r] + k);
#pragma unroll
              for (int w = 0; w < 8; ++w) {
                acc[r][w] = fmaf(-av.x, bv[w].x, acc[r][w]);
                acc[r][w] = fmaf(-av.y, bv[w].y, acc[r][w]);
                acc[r][w] = fmaf(-av.z, bv[w].z, acc[r][w]);
                acc[r][w] = fmaf(-av.w, bv[w].w, acc[r][w]);
              }
            }
          }
        }
        // 8 x 8 diagonal block (held by lanes 0..7, slot 0) and the rows below it
#pragma unroll
        for (int w = 0; w < 8; ++w) {
          float dw = __shfl_sync(FULL, acc[0][w], w);
          const int col = c0 + w;
          if (col < n) {
            if (!(dw > 0.f) || !isfinite(dw)) {
              bad = true;
              dw = 1.f;
            }
          } else {
            dw = 1.f;  // right-hand-side row and identity padding
          }
          const float rinv = rsqrtf(dw);
          if (lane == 0) invd[col] = rinv;
#pragma unroll
          for (int r = 0; r < NR; ++r)
            if (32 * r < rows_left) acc[r][w] *= rinv;
#pragma unroll
          for (int v = w + 1; v < 8; ++v) {
            const float lvw = __shfl_sync(FULL, acc[0][w], v);
#pragma unroll
            for (int r = 0; r < NR; ++r)
              if (32 * r < rows_left) acc[r][v] = fmaf(-acc[r][w], lvw, acc[r][v]);
          }
        }
#pragma unroll
        for (int r = 0; r < NR; ++r) {
          if (valid[r]) {
            *reinterpret_cast<float4*>(A + off[r] + c0) =
                make_float4(acc[r][0], acc[r][1], acc[r][2], acc[r][3]);
            *reinterpret_cast<float4*>(A + off[r] + c0 + 4) =
                make_float4(acc[r][4], acc[r][5], acc[r][6], acc[r][7]);
          }
        }
        __syncwarp();
      }
      if (bad) {
        if (lane == 0) report_error(&stats->status, THANOS_ERR_NOT_SPD, row);
        for (int jj = lane; jj < Bw; jj += 32) store_split3(D + (int64_t)row * ldd + jj, dplane, 0.f);
        __syncwarp();
        continue;
      }

      // ---- back substitution L^T x = y with y = row n of L, panels of 8 from the bottom;
      //      lane k & 31 (slot k / 32) owns x_k
      float* Arhs = A + tri_row_off(n);
      {
        float res[NR];
#pragma unroll
        for (int r = 0; r < NR; ++r) {
          const int k = lane + 32 * r;
          res[r] = (k < n) ? Arhs[k] : 0.f;
        }
        for (int c0 = (n - 1) & ~7; c0 >= 0; c0 -= 8) {
          const int slot = c0 >> 5;  // the slot that owns this panel's unknowns
          float rp = res[0];
#pragma unroll
          for (int r = 1; r < NR; ++r)
            if (slot == r) rp = res[r];
          const int kk = lane + 32 * slot;  // this lane's unknown in that slot
          float xw[8];
          const int goff = tri_row_off(c0);
          const int pstride = c0 + 12;
#pragma unroll
          for (int w = 7; w >= 0; --w) {
            const int i = c0 + w;
            float xi = 0.f;
            if (i < n) {  // warp-uniform
              xi = __shfl_sync(FULL, rp, i & 31) * invd[i];
              const float lik = A[goff + w * pstride + (kk < i ? kk : 0)];
              if (kk >= c0 && kk < i) rp = fmaf(-lik, xi, rp);
              if (kk == i) rp = xi;
            }
            xw[w] = xi;
          }
#pragma unroll
          for (int r = 0; r < NR; ++r) {
            if (slot == r) res[r] = rp;
            const int k = lane + 32 * r;
            if (32 * r < c0) {  // warp-uniform: this slot has unknowns left of the panel
              const int kc = k < c0 ? k : 0;
              float a8 = 0.f;
#pragma unroll
              for (int w = 0; w < 8; ++w) a8 = fmaf(A[goff + w * pstride + kc], xw[w], a8);
              if (k < c0) res[r] -= a8;
            }
          }
        }
        __syncwarp();
#pragma unroll
        for (int r = 0; r < NR; ++r) {
          const int k = lane + 32 * r;
          if (k < n) Arhs[k] = res[r];
          else if (k < n + 4) Arhs[k] = 0.f;  // the product below reads x in groups of four
        }
        __syncwarp();
      }

      // ---- delta over the block
      for (int a = lane; a < s; a += 32) dvec[qlist[a]] = -wblk[qlist[a]];
      if (kpath) {
        for (int e = lane; e < n; e += 32) dvec[sel[e]] = Arhs[e];
      } else {
        // delta_k = -sum_a lambda_a G[q_a, k_e]
        for (int e0 = 0; e0 < no; e0 += 32) {
          const int e = e0 + lane;
          const int col = (e < no) ? (int)oth[e] : 0;
          float g0 = 0.f, g1 = 0.f;
          for (int a = 0; a < n; a += 4) {
            const ushort4 ix = *reinterpret_cast<const ushort4*>(sel + a);
            const float4 xv = *reinterpret_cast<const float4*>(Arhs + a);
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

constexpr size_t SOLVE_SMEM_BUDGET = 227 * 1024;  // the most dynamic shared memory a CTA can get
constexpr int SOLVE_MAX_WARPS = 15;               // launch bound of solve_rows_fast_kernel
constexpr float UNCACHED_ROW_COST = 1.4f;         // time of a row without the shared copy of G / S over with it

template <int NR>
thanos_status_t launch_fast(float* Wc, const uint8_t* mask, const float* G, const float* S,
                            int ld_mat, __nv_bfloat16* D, int64_t dplane, int c, int b, int j1, int Bw,
                            int ldd, int n_max,
                            const int* row_lists, const unsigned* list_counts, int fixed_kind,
                            int report_max_s, thanos_stats_t* stats, cudaStream_t stream) {
  const int panels = (n_max + 1 + 7) / 8;
  // A warp works through its rows one after the other, and a row takes about the same time
  // whatever else is resident on the SM: a launch lasts (rows per warp, rounded up) x (time of a
  // row).  With G / S copied to shared memory a row is faster (33-35 us against 45-50 us at
  // B = 128, 50 %), but the copy leaves room for fewer warps; take whichever comes out shorter.
  const bool can_copy = (size_t)Bw * (Bw | 1) * 4 <= 72 * 1024;
  bool in_smem = false;
  int warps = 0;
  float best = 0.f;
  for (int copy = can_copy ? 1 : 0; copy >= 0; --copy) {
    const SolveSmemLayout l = solve_layout(Bw, panels, copy != 0);
    int wmax = (int)((SOLVE_SMEM_BUDGET - 4 * (size_t)l.mat_floats) / l.per_warp_bytes);
    if (wmax > SOLVE_MAX_WARPS) wmax = SOLVE_MAX_WARPS;
    for (int w = wmax; w >= 1 && w >= wmax - 1; --w) {
      const float cost = (float)ceil_div(c, (int64_t)NUM_SMS * w) * (copy ? 1.f : UNCACHED_ROW_COST);
      if (warps == 0 || cost < best || (cost == best && copy == 0 && !in_smem)) {
        best = cost;
        warps = w;
        in_smem = copy != 0;
      }
    }
  }
  if (warps < 1) return THANOS_ERR_SHAPE;
  SolveSmemLayout lay = solve_layout(Bw, panels, in_smem);
  const size_t smem = 4 * (size_t)lay.mat_floats + (size_t)warps * lay.per_warp_bytes;
  {
    static std::atomic<unsigned long long> done{0};
    THANOS_CUDA(ensure_max_dyn_smem(solve_rows_fast_kernel<NR>, (int)SOLVE_SMEM_BUDGET, done));
  }
  int64_t grid = ceil_div(c, warps);
  if (grid > NUM_SMS) grid = NUM_SMS;
  solve_rows_fast_kernel<NR><<<(unsigned)grid, warps * 32, smem, stream>>>(
      Wc, mask, G, S, ld_mat, D, dplane, c, b, j1, Bw, ldd, panels, in_smem ? 1 : 0, row_lists,
      list_counts, fixed_kind, report_max_s, stats);
  THANOS_CHECK_LAUNCH();
  return THANOS_OK;
}

}  // namespace

int tile_solve_max_unknowns();
thanos_status_t launch_tile_solve(float* Wc, const uint8_t* mask, const float* G, const float* S,
                                  int ld_mat, __nv_bfloat16* D, int64_t dplane, int c, int b,
                                  int j1, int Bw, int ldd, int n_max, const int* row_lists,
                                  const unsigned* list_counts, int fixed_kind, int report_max_s,
                                  thanos_stats_t* stats, cudaStream_t stream);
int cta_solve_max_unknowns();
thanos_status_t launch_cta_solve(float* Wc, const uint8_t* mask, const float* G, const float* S,
                                 int ld_mat, __nv_bfloat16* D, int64_t dplane, int c, int b, int j1,
                                 int Bw, int ldd, int n_max, const int* row_lists,
                                 const unsigned* list_counts, int fixed_kind, int report_max_s,
                                 thanos_stats_t* stats, cudaStream_t stream);

// Systems of up to 64 unknowns go to the warp-per-row tile kernel (solve_tile.cu), up to 159 to the
// warp-per-row panel kernel above, larger ones to the CTA-per-row kernel; n_small_max is the
// largest min(|q|, |k|) a row can have.
bool solve_supported(int s_direct_max, int n_small_max) {
  (void)s_direct_max;
  return n_small_max <= cta_solve_max_unknowns();
}

// Solves every row of the block [j1, j1 + Bw): writes the block's new weights into Wc and the
// change D (c x Bw as three bf16 planes dplane elements apart, leading dimension ldd).  G and S are the block's Bw x Bw matrices (leading
// dimension ld_mat).  s_fixed >= 0 says every row removes exactly s_fixed entries (n:m);
// otherwise row_lists[2][c] / list_counts[2] hold the rows sorted by kind (0: |q| <= |k|).
thanos_status_t launch_block_solve(float* Wc, const uint8_t* mask, const float* G, const float* S,
                                   int ld_mat, __nv_bfloat16* D, int64_t dplane, int c, int b, int j1,
                                   int Bw, int ldd, int s_fixed, const int* row_lists,
                                   const unsigned* list_counts,
                                   thanos_stats_t* stats, cudaStream_t stream) {
  const bool uniform = s_fixed >= 0;
  const int n_small = uniform ? (s_fixed < Bw - s_fixed ? s_fixed : Bw - s_fixed) : Bw / 2;
  const int fixed_kind = uniform ? (s_fixed > Bw - s_fixed ? 1 : 0) : 0;
  const int* rl = uniform ? nullptr : row_lists;
  const unsigned* lc = uniform ? nullptr : list_counts;
  const int rep = uniform ? 1 : 0;
  // 97 to 159 unknowns in a block of at most 256 columns: the four-warp CTAs of solve_cta.cu
  // keep four rows per SM in flight, the warp-per-row kernel (41 KB per warp) only five warps
  if (n_small + 1 > 160 || (n_small + 1 > 96 && Bw <= 256))
    return launch_cta_solve(Wc, mask, G, S, ld_mat, D, dplane, c, b, j1, Bw, ldd, n_small, rl, lc,
                            fixed_kind, rep, stats, stream);
  // up to 64 unknowns: the warp-per-row tile kernel with tensor-core trailing updates
  if (n_small <= tile_solve_max_unknowns() && Bw <= 1024)
    return launch_tile_solve(Wc, mask, G, S, ld_mat, D, dplane, c, b, j1, Bw, ldd, n_small, rl, lc,
                             fixed_kind, rep, stats, stream);
  if (n_small + 1 <= 32)
    return launch_fast<1>(Wc, mask, G, S, ld_mat, D, dplane, c, b, j1, Bw, ldd, n_small, rl, lc,
                          fixed_kind, rep, stats, stream);
  if (n_small + 1 <= 64)
    return launch_fast<2>(Wc, mask, G, S, ld_mat, D, dplane, c, b, j1, Bw, ldd, n_small, rl, lc,
                          fixed_kind, rep, stats, stream);
  if (n_small + 1 <= 96)
    return launch_fast<3>(Wc, mask, G, S, ld_mat, D, dplane, c, b, j1, Bw, ldd, n_small, rl, lc,
                          fixed_kind, rep, stats, stream);
  return launch_fast<5>(Wc, mask, G, S, ld_mat, D, dplane, c, b, j1, Bw, ldd, n_small, rl, lc,
                        fixed_kind, rep, stats, stream);
}

}  // namespace thanos
