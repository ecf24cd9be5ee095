// The block sweep of Algorithm 1 (unstructured) and Algorithm 4 (n:m, alpha = 0):
// per block of B columns -- metric, mask, per-row solve, update of all columns to the right.
//
// With U from thanos_prepare_inverse (U^T U = inv(H_d), upper) the residual inverse of a block
// starting at j1 is U[j1:, j1:]^T U[j1:, j1:].  Per block, with U_bb = U[j1:j2, j1:j2] and
// V_bb = inv(U_bb):
//   G = U_bb^T U_bb      the block of the residual inverse (R-hat = G[q, q] in Eqs. 5-7),
//   S = V_bb V_bb^T      its inverse, for rows that remove more than half of the block,
//   P2 = V_bb U[j1:j2, j2:]
// and Eq. 8 splits into the change of the block itself, delta (c x B, from the per-row solves;
// delta_q = -w_q), and the change of every column to the right, which is the dense product
//   W[:, j2:] += delta P2      (because -lambda-hat R = delta inv(G) (U_bb^T U[j1:j2, j1:])).
// G, S, V_bb and P2 depend only on U, so they are computed for all blocks at the start of the
// sweep.
#include <cooperative_groups.h>

#include "simt_gemm.cuh"
#include "tc_gemm.cuh"

namespace thanos {

bool solve_supported(int s_direct_max, int n_small_max);
thanos_status_t launch_block_solve(float* Wc, const uint8_t* mask, const float* G, const float* S,
                                   int ld_mat, __nv_bfloat16* D, int64_t dplane, int c, int b, int j1,
                                   int Bw, int ldd, int s_fixed, const int* row_lists,
                                   const unsigned* list_counts,
                                   thanos_stats_t* stats, cudaStream_t stream);

namespace {

// Selection of the block threshold: the r-th smallest metric key over the residual (Eq. psi with
// the running budget r of Algorithm 1).  Keys are the fp32 bit patterns of |w| * ||X_j|| (>= 0, so
// they order like the values).  Two routes, both exact:
//   bracket  the threshold moves little from block to block, so one pass counts the keys below a
//            window of 2^16 key values around the previous threshold, bins the keys inside it
//            (512 bins of 128 values) and copies them out (about 1 in 130); a second, short pass
//            over the copied keys resolves the 512 values of the hit bin;
//   radix    four passes over 8, 8, 8 and 7 key bits (first block, or when the window misses).
// One pass body does whichever pass the sweep state asks for; the last CTA to finish a pass reads
// the histogram, decides and sets the next phase.  Per block it runs once as a kernel of its own
// (the pass over the residual) and then inside one cooperative launch, behind grid barriers, as
// often as the route still needs.
constexpr int HIST_BINS = 512;
constexpr int RADIX_BINS = 256;
constexpr int RADIX_REPL = 8;           // shared-memory copies of a radix histogram (by lane & 7)
constexpr int WINDOW_LOG2 = 16;        // key values covered by the bracket: 2^16 (0.8 % of a binade),
constexpr int WINDOW_LOG2_WIDE = 18;   // 2^18 for the rest of a sweep once a bracket has missed
constexpr int WINDOW_BINS_LOG2 = 9;    // 512 bracket bins
constexpr int CTA_CAND = 6144;          // keys inside the window one CTA can hold before copying out
__host__ __device__ constexpr int pass_bits(int pass) { return pass == 3 ? 7 : 8; }
__host__ __device__ constexpr int pass_shift(int pass) { return pass == 0 ? 23 : (pass == 1 ? 15 : (pass == 2 ? 7 : 0)); }

enum SelectPhase : int {
  PH_RADIX0 = 0, PH_RADIX1 = 1, PH_RADIX2 = 2, PH_RADIX3 = 3, PH_BRACKET = 4, PH_REFINE = 5,
  PH_DONE = 6
};

struct SweepState {
  long long r;                   // removals still to place before the current block
  unsigned long long k_rem;      // rank still to resolve inside the current candidate range
  unsigned long long need_eq;    // how many entries with key == tau are removed
  unsigned long long count_eq;   // how many entries with key == tau the residual holds
  unsigned long long blk_count;  // entries removed in the current block
  unsigned long long below;      // bracket pass: keys below the window
  unsigned int prefix;           // radix: key bits fixed so far
  unsigned int tau;              // threshold key of the current block
  unsigned int lo;               // start of the bracket window / of the bin being refined
  unsigned int tau_prev;         // threshold of the previous block
  int have_prev;
  int none;                      // nothing to remove in this block
  int phase;                     // what the next select pass does
  unsigned int ticket;           // CTAs that have finished the current pass
  unsigned int mark_ticket;      // same for the mask kernel
  unsigned int cand_total;       // keys the bracket pass copied out of its window
  int cand_overflow;             // the copy did not fit: the refine pass rescans the residual
  int wide;                      // a bracket missed in this sweep: use the wide window
  int tie_in_block;              // an entry equal to the threshold lies in the current block's columns
};

__device__ __forceinline__ unsigned metric_key(float w, float xn) {
  // |w| * ||X_j|| in fp32; non-negative floats order like their bit patterns
  return __float_as_uint(fabsf(w) * xn);
}

// ------------------------------------------------------------------ per-block matrices
// Dense copy of U_bb (zeros below the diagonal) and V_bb = inv(U_bb).  Grid (strips of 64
// columns, blocks): a CTA owns 64 columns of V_bb and solves U_bb V = I for them by blocked back
// substitution over row blocks of 32 from the bottom: the finished rows of its strip stay in
// shared memory, the product with the U tiles to their right and the 32 x 32 triangular solve
// are accumulated in double.
constexpr int INV_STRIP = 64;
constexpr int INV_RB = 32;

__host__ __device__ inline size_t block_inverse_smem(int B) {
  const size_t rows = (size_t)(B + INV_RB - 1) / INV_RB * INV_RB;
  return rows * INV_STRIP * sizeof(float) + INV_RB * INV_STRIP * sizeof(double) +
         INV_RB * (INV_RB + 1) * sizeof(float);
}

__global__ void __launch_bounds__(256)
block_inverse_kernel(const float* __restrict__ U, float* __restrict__ Ubb, float* __restrict__ Vbb,
                     int b, int B) {
  extern __shared__ __align__(16) unsigned char inv_dyn[];
  double* Rs = reinterpret_cast<double*>(inv_dyn);                       // [32][64]
  float* Vs = reinterpret_cast<float*>(Rs + INV_RB * INV_STRIP);         // [B rounded up to 32][64]
  float* Ut = Vs + (size_t)((B + INV_RB - 1) / INV_RB * INV_RB) * INV_STRIP;  // [32][33]
  const int tid = threadIdx.x;
  const int bb = blockIdx.y;
  const int c0 = blockIdx.x * INV_STRIP;
  const int j1 = bb * B;
  const int Bw = (b - j1 < B) ? b - j1 : B;
  float* Uo = Ubb + (size_t)bb * B * B;
  float* Vo = Vbb + (size_t)bb * B * B;
  const float* Ub = U + (int64_t)j1 * b + j1;
  for (int e = tid; e < B * INV_STRIP; e += 256) {
    const int i = e / INV_STRIP, j = c0 + (e % INV_STRIP);
    if (j >= B) continue;
    float u = 0.f;
    if (i < Bw && j < Bw && j >= i) u = Ub[(int64_t)i * b + j];
    Uo[(size_t)i * B + j] = u;
  }
  const int rows_tot = (c0 + INV_STRIP < Bw) ? c0 + INV_STRIP : Bw;  // rows that can be non-zero
  const int nI = rows_tot > 0 && c0 < Bw ? (rows_tot + INV_RB - 1) / INV_RB : 0;
  const int col = tid & (INV_STRIP - 1), rg = tid >> 6;  // rows rg, rg + 4, ... of a row block
  for (int I = nI - 1; I >= 0; --I) {
    const int r0 = I * INV_RB;
    double acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0.0;
    for (int K = I + 1; K < nI; ++K) {
      __syncthreads();
      for (int e = tid; e < INV_RB * INV_RB; e += 256) {
        const int r = e >> 5, kk = e & 31;
        const int gi = r0 + r, gk = K * INV_RB + kk;
        Ut[r * (INV_RB + 1) + kk] = (gi < Bw && gk < Bw) ? Ub[(int64_t)gi * b + gk] : 0.f;
      }
      __syncthreads();
#pragma unroll 4
      for (int kk = 0; kk < INV_RB; ++kk) {
        const double v = (double)Vs[(size_t)(K * INV_RB + kk) * INV_STRIP + col];
#pragma unroll
        for (int i = 0; i < 8; ++i)
          acc[i] = fma((double)Ut[(rg + 4 * i) * (INV_RB + 1) + kk], v, acc[i]);
      }
    }
    __syncthreads();
    for (int e = tid; e < INV_RB * INV_RB; e += 256) {
      const int r = e >> 5, kk = e & 31;
      const int gi = r0 + r, gk = r0 + kk;
      Ut[r * (INV_RB + 1) + kk] = (gi < Bw && gk < Bw && gk >= gi) ? Ub[(int64_t)gi * b + gk] : 0.f;
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int r = rg + 4 * i;
      Rs[r * INV_STRIP + col] = ((r0 + r == c0 + col) ? 1.0 : 0.0) - acc[i];
    }
    __syncthreads();
    if (tid < INV_STRIP) {
      for (int r = INV_RB - 1; r >= 0; --r) {
        double x = 0.0;
        if (r0 + r < rows_tot) {
          x = Rs[r * INV_STRIP + col];
          for (int k = r + 1; k < INV_RB; ++k)
            x = fma(-(double)Ut[r * (INV_RB + 1) + k], Rs[k * INV_STRIP + col], x);
          x /= (double)Ut[r * (INV_RB + 1) + r];
        }
        Rs[r * INV_STRIP + col] = x;
        Vs[(size_t)(r0 + r) * INV_STRIP + col] = (float)x;
      }
    }
  }
  __syncthreads();
  for (int e = tid; e < B * INV_STRIP; e += 256) {
    const int i = e / INV_STRIP, jj = e % INV_STRIP;
    if (c0 + jj >= B) continue;
    Vo[(size_t)i * B + c0 + jj] = (i < nI * INV_RB && i < B) ? Vs[(size_t)i * INV_STRIP + jj] : 0.f;
  }
}

// which = 0: G = U_bb^T U_bb;  which = 1: S = V_bb V_bb^T.  Grid (B/64, B/64, blocks).
template <int WHICH>
__global__ void __launch_bounds__(256)
block_gram_kernel(const float* __restrict__ Fbb, float* __restrict__ Out, int b, int B) {
  using G = SimtGemm<64, 64, 16, 4, 4, WHICH == 0, WHICH == 1, float, float>;
  __shared__ float smem[G::SMEM_FLOATS];
  const int bb = blockIdx.z;
  const int j1 = bb * B;
  const int Bw = (b - j1 < B) ? b - j1 : B;
  const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
  if (m0 >= Bw || n0 >= Bw) return;
  const float* F = Fbb + (size_t)bb * B * B;
  float acc[4][4] = {};
  G::run(F, B, F, B, Bw, Bw, m0, n0, 0, Bw, acc, smem);
  float* O = Out + (size_t)bb * B * B;
  const int tx = threadIdx.x % G::TX, ty = threadIdx.x / G::TX;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int gm = m0 + G::row_of(ty, i);
    if (gm >= Bw) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int gn = n0 + G::col_of(tx, j);
      if (gn < Bw) O[(size_t)gm * B + gn] = acc[i][j];
    }
  }
}

// P2[j1 + m, j2 + n] = sum_k V_bb[m, k] U[j1 + k, j2 + n] for every block.  Grid (n tiles of the
// widest block, B/64, blocks).
__global__ void __launch_bounds__(256)
block_rows_kernel(const float* __restrict__ U, const float* __restrict__ Vbb,
                  __nv_bfloat16* __restrict__ P2, int b, int B) {
  using G = SimtGemm<64, 64, 16, 4, 4, false, false, float, float>;
  __shared__ float smem[G::SMEM_FLOATS];
  const int bb = blockIdx.z;
  const int j1 = bb * B;
  const int Bw = (b - j1 < B) ? b - j1 : B;
  const int j2 = j1 + Bw;
  const int N = b - j2;
  const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
  if (m0 >= Bw || n0 >= N) return;
  float acc[4][4] = {};
  // V_bb is upper-triangular: column k contributes to rows m <= k
  G::run(Vbb + (size_t)bb * B * B, B, U + (int64_t)j1 * b + j2, b, Bw, N, m0, n0, m0, Bw, acc,
         smem);
  const int tx = threadIdx.x % G::TX, ty = threadIdx.x / G::TX;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int gm = m0 + G::row_of(ty, i);
    if (gm >= Bw) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int gn = n0 + G::col_of(tx, j);
      if (gn < N) {
        float v = acc[i][j];
        __nv_bfloat16* o = P2 + (int64_t)(j1 + gm) * b + j2 + gn;
#pragma unroll
        for (int pl = 0; pl < 3; ++pl) {  // three bf16 planes of the fp32 value
          const __nv_bfloat16 hb = __float2bfloat16_rn(v);
          o[(int64_t)pl * b * b] = hb;
          v -= __bfloat162float(hb);
        }
      }
    }
  }
}

// ------------------------------------------------------------------ unstructured selection
// Warp scan over NBIN (<= 512) histogram bins: finds the bin that holds rank k (1-based) and
// returns (bin, entries before it, entries in it) to every lane; bin = -1 if k is out of range.
__device__ __forceinline__ void find_rank_bin(const unsigned* hist, int nbin, unsigned long long k,
                                              int& bin_out, unsigned long long& before_out,
                                              unsigned long long& inbin_out) {
  const int lane = threadIdx.x & 31;
  constexpr int PER = HIST_BINS / 32;
  unsigned long long loc[PER];
  unsigned long long tsum = 0;
#pragma unroll
  for (int e = 0; e < PER; ++e) {
    const int bin = lane * PER + e;
    loc[e] = bin < nbin ? (unsigned long long)__ldcg(&hist[bin]) : 0ull;
    tsum += loc[e];
  }
  unsigned long long inc = tsum;
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned long long v = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += v;
  }
  unsigned long long excl = inc - tsum;
  int found = -1;
  unsigned long long fb = 0, fi = 0;
#pragma unroll
  for (int e = 0; e < PER; ++e) {
    if (found < 0 && k > excl && k <= excl + loc[e]) {
      found = lane * PER + e;
      fb = excl;
      fi = loc[e];
    }
    excl += loc[e];
  }
  const unsigned has = __ballot_sync(0xffffffffu, found >= 0);
  if (has == 0) {
    bin_out = -1;
    before_out = inbin_out = 0;
    return;
  }
  const int src = __ffs(has) - 1;
  bin_out = __shfl_sync(0xffffffffu, found, src);
  before_out = __shfl_sync(0xffffffffu, fb, src);
  inbin_out = __shfl_sync(0xffffffffu, fi, src);
}

// One pass of the threshold selection over the residual W[:, j1:]; what it does is st->phase.
// Shared histogram: radix passes keep one counter per (bin, lane) -- a warp never hits the same
// bank twice, whatever the skew of the metric; bracket / refine passes see few keys inside
// their range and use plain counters.
template <int BR_UNROLL>
__device__ __forceinline__ void select_pass_body(const float* __restrict__ Wc,
                                                 const float* __restrict__ xnorm, int c, int b, int j1,
                                                 SweepState* st, unsigned* __restrict__ hist,
                                                 const int64_t* r_ext,
                                                 unsigned* __restrict__ list_counts, int first_launch,
                                                 thanos_stats_t* stats, unsigned* __restrict__ cand,
                                                 unsigned cand_cap) {
  __shared__ unsigned sh[RADIX_BINS * RADIX_REPL];
  __shared__ unsigned s_cand[CTA_CAND];
  __shared__ unsigned s_ncand, s_cbase;
  __shared__ int s_last;
  __shared__ unsigned s_below;
  const int phase = *reinterpret_cast<volatile int*>(&st->phase);
  if (phase == PH_DONE && !first_launch) return;
  if (first_launch && blockIdx.x == 0 && threadIdx.x == 0) {
    list_counts[0] = list_counts[1] = 0;
    st->tie_in_block = 0;
    if (r_ext) st->r = *r_ext;
  }
  const int lane = threadIdx.x & 31;
  const int w4 = (b - j1) >> 2;
  const float4* xr = reinterpret_cast<const float4*>(xnorm + j1);
  const bool radix = phase <= PH_RADIX3;
  const int nclear = radix ? RADIX_BINS * RADIX_REPL : HIST_BINS;
  for (int i = threadIdx.x; i < nclear; i += 256) sh[i] = 0;
  if (threadIdx.x == 0) {
    s_below = 0;
    s_ncand = 0;
  }
  __syncthreads();
  unsigned below = 0;
  if (radix) {
    const int shift = pass_shift(phase), bits = pass_bits(phase);
    const unsigned prefix = st->prefix;
    const unsigned bmask = (1u << bits) - 1u;
    for (int row = blockIdx.x; row < c; row += gridDim.x) {
      const float4* wr = reinterpret_cast<const float4*>(Wc + (int64_t)row * b + j1);
      for (int q0 = threadIdx.x; q0 < w4; q0 += 4 * 256) {
        float4 w[4], x[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {  // four loads in flight per thread
          const int q = q0 + u * 256;
          w[u] = q < w4 ? wr[q] : make_float4(0.f, 0.f, 0.f, 0.f);
          x[u] = q < w4 ? __ldg(&xr[q]) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          if (q0 + u * 256 >= w4) break;
          const unsigned k[4] = {metric_key(w[u].x, x[u].x), metric_key(w[u].y, x[u].y),
                                 metric_key(w[u].z, x[u].z), metric_key(w[u].w, x[u].w)};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            if (phase == PH_RADIX0 || (k[e] >> (shift + bits)) == prefix)
              atomicAdd(&sh[((k[e] >> shift) & bmask) * RADIX_REPL + (lane & (RADIX_REPL - 1))], 1u);
          }
        }
      }
    }
  } else if (phase == PH_REFINE && !st->cand_overflow) {
    // the bracket pass copied every key of its window out: only those are looked at again
    const unsigned lo = st->lo;
    const unsigned total = st->cand_total;
    for (unsigned i = blockIdx.x * 256u + threadIdx.x; i < total; i += gridDim.x * 256u) {
      const unsigned d = __ldcg(&cand[i]) - lo;
      if (d < (unsigned)HIST_BINS) atomicAdd(&sh[d], 1u);
    }
  } else if (phase == PH_BRACKET) {
    // The hot pass: per element one multiply, one compare-and-count, one window test; keys inside
    // the window (about 1 in 130) take the slow path that bins and copies them.
    const unsigned lo = st->lo;
    const int wlog = st->wide ? WINDOW_LOG2_WIDE : WINDOW_LOG2;
    const unsigned WINDOW = 1u << wlog;
    const int WINDOW_SHIFT = wlog - WINDOW_BINS_LOG2;
    // The residual is walked as one list of c * w4 16-byte items (row-major), 256 consecutive
    // items per CTA and step, so that every thread has a load to issue whatever the width of the
    // residual; a thread's (row, q) advances by the grid's stride without a division.
    // BR_UNROLL loads in flight per thread: two when the working copy sits in L2, four when the
    // residual streams from HBM.
    const unsigned stride = gridDim.x * 256u;
    const unsigned first = blockIdx.x * 256u + threadIdx.x;
    const unsigned d_row = stride / (unsigned)w4, d_q = stride - d_row * (unsigned)w4;
    unsigned row = first / (unsigned)w4, q = first - row * (unsigned)w4;
    while (row < (unsigned)c) {
      float4 wv[BR_UNROLL], xv[BR_UNROLL];
      bool ok[BR_UNROLL];
#pragma unroll
      for (int u = 0; u < BR_UNROLL; ++u) {
        ok[u] = row < (unsigned)c;
        wv[u] = make_float4(0.f, 0.f, 0.f, 0.f);
        xv[u] = wv[u];
        if (ok[u]) {
          wv[u] = reinterpret_cast<const float4*>(Wc + (int64_t)row * b + j1)[q];
          xv[u] = __ldg(&xr[q]);
        }
        row += d_row;
        q += d_q;
        if (q >= (unsigned)w4) {
          q -= (unsigned)w4;
          ++row;
        }
      }
#pragma unroll
      for (int u = 0; u < BR_UNROLL; ++u) {
        if (!ok[u]) break;
        const float4 w = wv[u];
        const float4 x = xv[u];
        const unsigned k0 = metric_key(w.x, x.x), k1 = metric_key(w.y, x.y);
        const unsigned k2 = metric_key(w.z, x.z), k3 = metric_key(w.w, x.w);
        below += (k0 < lo) + (k1 < lo) + (k2 < lo) + (k3 < lo);
        // k - lo wraps to a huge value for k < lo, so one unsigned test finds the window
        const unsigned d0 = k0 - lo, d1 = k1 - lo, d2 = k2 - lo, d3 = k3 - lo;
        if ((d0 < WINDOW) | (d1 < WINDOW) | (d2 < WINDOW) | (d3 < WINDOW)) {
          const unsigned kk[4] = {k0, k1, k2, k3};
          const unsigned dd[4] = {d0, d1, d2, d3};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            if (dd[e] < WINDOW) {
              atomicAdd(&sh[dd[e] >> WINDOW_SHIFT], 1u);
              const unsigned pos = atomicAdd(&s_ncand, 1u);
              if (pos < (unsigned)CTA_CAND) s_cand[pos] = kk[e];
            }
          }
        }
      }
    }
  } else {
    // refine over the whole residual (only when the copied keys did not fit)
    const unsigned lo = st->lo;
    for (int row = blockIdx.x; row < c; row += gridDim.x) {
      const float4* wr = reinterpret_cast<const float4*>(Wc + (int64_t)row * b + j1);
      for (int q = threadIdx.x; q < w4; q += 256) {
        const float4 w = wr[q];
        const float4 x = __ldg(&xr[q]);
        const unsigned k[4] = {metric_key(w.x, x.x), metric_key(w.y, x.y), metric_key(w.z, x.z),
                               metric_key(w.w, x.w)};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const unsigned d = k[e] - lo;
          if (d < (unsigned)HIST_BINS) atomicAdd(&sh[d], 1u);
        }
      }
    }
  }
  __syncthreads();
  if (radix) {
    const int nbin = 1 << pass_bits(phase);
    for (int bin = threadIdx.x; bin < nbin; bin += 256) {
      unsigned t = 0;
#pragma unroll
      for (int l = 0; l < RADIX_REPL; ++l) t += sh[bin * RADIX_REPL + l];
      if (t) atomicAdd(&hist[bin], t);
    }
  } else {
    for (int bin = threadIdx.x; bin < HIST_BINS; bin += 256)
      if (sh[bin]) atomicAdd(&hist[bin], sh[bin]);
    if (phase == PH_BRACKET) {
      for (int o = 16; o > 0; o >>= 1) below += __shfl_down_sync(0xffffffffu, below, o);
      if (lane == 0 && below) atomicAdd(&s_below, below);
      __syncthreads();
      const unsigned ncand = s_ncand;
      if (threadIdx.x == 0) {
        if (s_below) atomicAdd(&st->below, (unsigned long long)s_below);
        if (ncand > (unsigned)CTA_CAND) {
          st->cand_overflow = 1;
          s_cbase = cand_cap;
        } else {
          s_cbase = ncand ? atomicAdd(&st->cand_total, ncand) : 0u;
          if (ncand && s_cbase + ncand > cand_cap) st->cand_overflow = 1;
        }
      }
      __syncthreads();
      const unsigned cbase = s_cbase;
      if (ncand <= (unsigned)CTA_CAND && cbase + ncand <= cand_cap)
        for (unsigned i = threadIdx.x; i < ncand; i += 256) cand[cbase + i] = s_cand[i];
    }
  }
  // ---- the last CTA to get here decides
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) s_last = (atomicAdd(&st->ticket, 1u) == gridDim.x - 1) ? 1 : 0;
  __syncthreads();
  if (!s_last || threadIdx.x >= 32) return;
  __threadfence();
  volatile SweepState* vs = st;
  const unsigned* vh = hist;
  int next = PH_DONE;
  if (first_launch) {
    const long long r = vs->r;
    if (lane == 0) {
      st->none = r <= 0 ? 1 : 0;
      st->k_rem = r > 0 ? (unsigned long long)r : 0ull;
      st->blk_count = 0;
      st->need_eq = 0;
      st->count_eq = 0;
    }
    __syncwarp();
  }
  const bool none = vs->none != 0;
  const unsigned long long k = vs->k_rem;
  if (none) {
    next = PH_DONE;
  } else if (radix) {
    int bin;
    unsigned long long before, inbin;
    find_rank_bin(const_cast<const unsigned*>(vh), 1 << pass_bits(phase), k, bin, before, inbin);
    if (bin < 0) bin = 0;  // cannot happen: k <= number of candidates
    const unsigned np = (vs->prefix << pass_bits(phase)) | (unsigned)bin;
    if (lane == 0) {
      st->prefix = phase == PH_RADIX3 ? 0u : np;
      st->k_rem = k - before;
      if (phase == PH_RADIX3) {
        st->tau = np;
        st->need_eq = k - before;
        st->count_eq = inbin;
      }
    }
    next = phase == PH_RADIX3 ? PH_DONE : phase + 1;
  } else if (phase == PH_BRACKET) {
    const unsigned long long bel = vs->below;
    int bin = -1;
    unsigned long long before = 0, inbin = 0;
    if (k > bel) find_rank_bin(const_cast<const unsigned*>(vh), HIST_BINS, k - bel, bin, before, inbin);
    if (bin >= 0) {
      if (lane == 0) {
        st->lo = vs->lo + ((unsigned)bin << ((vs->wide ? WINDOW_LOG2_WIDE : WINDOW_LOG2) - WINDOW_BINS_LOG2));
        st->k_rem = k - bel - before;
        if (vs->cand_overflow) stats->select_rescans += 1;
      }
      next = PH_REFINE;
    } else {
      if (lane == 0) {
        st->prefix = 0;
        st->wide = 1;
        stats->select_misses += 1;
      }
      next = PH_RADIX0;  // the window missed: full radix select, k_rem is still the rank
    }
  } else {  // PH_REFINE
    int bin;
    unsigned long long before, inbin;
    find_rank_bin(const_cast<const unsigned*>(vh), HIST_BINS, k, bin, before, inbin);
    if (bin < 0) bin = 0;  // cannot happen: the bracket pass counted this bin
    if (lane == 0) {
      st->tau = vs->lo + (unsigned)bin;
      st->need_eq = k - before;
      st->count_eq = inbin;
    }
    next = PH_DONE;
  }
  __syncwarp();
  for (int i = lane; i < HIST_BINS; i += 32) hist[i] = 0;
  if (lane == 0) {
    st->below = 0;
    st->ticket = 0;
    st->phase = next;
    if (next != PH_REFINE) {  // the copied keys are only needed by the refine pass
      st->cand_total = 0;
      st->cand_overflow = 0;
    }
  }
}

template <int BR_UNROLL>
__global__ void __launch_bounds__(256)
select_pass_kernel(const float* __restrict__ Wc, const float* __restrict__ xnorm, int c, int b,
                   int j1, SweepState* st, unsigned* __restrict__ hist, const int64_t* r_ext,
                   unsigned* __restrict__ list_counts, int first_launch, thanos_stats_t* stats,
                   unsigned* __restrict__ cand, unsigned cand_cap) {
  select_pass_body<BR_UNROLL>(Wc, xnorm, c, b, j1, st, hist, r_ext, list_counts, first_launch, stats,
                              cand, cand_cap);
}

// Rows' counts of entries equal to the threshold over the residual (only needed when the
// tie-break has to leave some of them unpruned and one of them lies in the block): a CTA takes
// rows blockIdx.x, blockIdx.x + gridDim.x, ...  256 threads per CTA.
__device__ __forceinline__ void tie_count_rows(const float* __restrict__ Wc,
                                               const float* __restrict__ xnorm, int c, int b, int j1,
                                               unsigned tau, unsigned* __restrict__ rowcnt) {
  __shared__ unsigned red[8];
  const int w4 = (b - j1) >> 2;
  for (int row = blockIdx.x; row < c; row += gridDim.x) {
    const float4* wr = reinterpret_cast<const float4*>(Wc + (int64_t)row * b + j1);
    const float4* xr = reinterpret_cast<const float4*>(xnorm + j1);
    unsigned cnt = 0;
#pragma unroll 4
    for (int q = threadIdx.x; q < w4; q += 256) {
      float4 w = wr[q];
      float4 x = __ldg(&xr[q]);
      cnt += (metric_key(w.x, x.x) == tau) + (metric_key(w.y, x.y) == tau) +
             (metric_key(w.z, x.z) == tau) + (metric_key(w.w, x.w) == tau);
    }
    for (int o = 16; o > 0; o >>= 1) cnt += __shfl_down_sync(0xffffffffu, cnt, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = cnt;
    __syncthreads();
    if (threadIdx.x == 0) {
      unsigned t = 0;
      for (int i = 0; i < 8; ++i) t += red[i];
      rowcnt[row] = t;
    }
    __syncthreads();
  }
}

// rowbase[row] = number of tied entries in the rows before it (exclusive scan by one CTA of 256).
__device__ __forceinline__ void tie_scan_rows(int c, const unsigned* __restrict__ rowcnt,
                                              unsigned long long* __restrict__ rowbase) {
  __shared__ unsigned long long wsum[8];
  __shared__ unsigned long long carry;
  if (threadIdx.x == 0) carry = 0;
  __syncthreads();
  for (int base = 0; base < c; base += 256) {
    const int row = base + threadIdx.x;
    const unsigned long long v = row < c ? __ldcg(&rowcnt[row]) : 0;
    unsigned long long inc = v;
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned long long u = __shfl_up_sync(0xffffffffu, inc, o);
      if ((threadIdx.x & 31) >= o) inc += u;
    }
    if ((threadIdx.x & 31) == 31) wsum[threadIdx.x >> 5] = inc;
    __syncthreads();
    unsigned long long before = carry;
    for (int w = 0; w < (int)(threadIdx.x >> 5); ++w) before += wsum[w];
    const unsigned long long excl = before + inc - v;
    if (row < c) rowbase[row] = excl;
    __syncthreads();
    if (threadIdx.x == 255) carry = excl + v;
    __syncthreads();
  }
}

// Everything a block's selection needs after its pass over the residual, in ONE cooperative launch
// with a grid barrier between the steps: the refine pass over the copied keys (the usual case), or
// up to four radix passes (three after a first radix pass, four after a bracket that missed).
// Last it finds out whether the order of tied entries can matter to this block's mask at all,
// and ranks them if so.
template <int BR_UNROLL>
__global__ void __launch_bounds__(256)
select_rest_kernel(const float* __restrict__ Wc, const float* __restrict__ xnorm, int c, int b,
                   int j1, int Bw, SweepState* st, unsigned* __restrict__ hist,
                   unsigned* __restrict__ list_counts, thanos_stats_t* stats,
                   unsigned* __restrict__ cand, unsigned cand_cap,
                   unsigned* __restrict__ rowcnt, unsigned long long* __restrict__ rowbase) {
  cooperative_groups::grid_group grid = cooperative_groups::this_grid();
  for (int it = 0; it < 4; ++it) {
    // the phase only changes between two grid barriers, so every CTA reads the same value
    if (*reinterpret_cast<volatile int*>(&st->phase) == PH_DONE) break;
    select_pass_body<BR_UNROLL>(Wc, xnorm, c, b, j1, st, hist, nullptr, list_counts, 0, stats, cand,
                                cand_cap);
    grid.sync();
  }
  // The threshold is final.  When only some of the entries equal to it are removed, their order
  // over the whole residual decides which -- but that only matters to this block's mask if one
  // of them lies in the block's own columns.  Look there (c * Bw entries) before anyone counts
  // ties over the whole residual.
  volatile SweepState* vs = st;
  if (vs->none || vs->need_eq == vs->count_eq) return;
  const unsigned tau = vs->tau;
  const int w4 = Bw >> 2;
  const float4* xr = reinterpret_cast<const float4*>(xnorm + j1);
  int found = 0;
  const unsigned total = (unsigned)c * (unsigned)w4;
  for (unsigned i = blockIdx.x * 256u + threadIdx.x; i < total; i += gridDim.x * 256u) {
    const unsigned row = i / (unsigned)w4, q = i - row * (unsigned)w4;
    const float4 w = reinterpret_cast<const float4*>(Wc + (int64_t)row * b + j1)[q];
    const float4 x = __ldg(&xr[q]);
    found |= (metric_key(w.x, x.x) == tau) | (metric_key(w.y, x.y) == tau) |
             (metric_key(w.z, x.z) == tau) | (metric_key(w.w, x.w) == tau);
  }
  if (__syncthreads_or(found) && threadIdx.x == 0) st->tie_in_block = 1;
  grid.sync();
  if (!vs->tie_in_block) return;
  // It does: rank the tied entries in (row, column) order -- their count per row over the whole
  // residual, then the exclusive scan over the rows that the mask kernel reads.
  tie_count_rows(Wc, xnorm, c, b, j1, tau, rowcnt);
  grid.sync();
  if (blockIdx.x == 0) tie_scan_rows(c, rowcnt, rowbase);
}

// One warp per row: set the block's mask bytes.  key < tau -> removed; key == tau -> removed
// while the (row, column)-ordered rank of the tie is below need_eq.
constexpr int MARK_WARPS = 32;  // rows per CTA and round of the mask kernel
__global__ void __launch_bounds__(32 * MARK_WARPS)
mark_block_kernel(const float* __restrict__ Wc, const float* __restrict__ xnorm,
                  uint8_t* __restrict__ mask, int c, int b, int j1, int Bw, SweepState* st,
                  const unsigned long long* __restrict__ rowbase, int* __restrict__ row_lists,
                  unsigned* __restrict__ list_counts, thanos_stats_t* stats, int64_t* r_ext) {
  __shared__ int s_last;
  // the rows of one round of the CTA (one per warp) by kind: the two row lists grow by one
  // atomic per kind and round instead of one per row
  __shared__ int s_rows[2][MARK_WARPS];
  __shared__ unsigned s_cnt[2], s_base[2];
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const bool none = st->none != 0;
  const unsigned tau = st->tau;
  const bool all_ties = st->need_eq == st->count_eq;
  const bool tie_in_block = st->tie_in_block != 0;  // else no entry of the block equals the threshold
  const unsigned long long need = st->need_eq;
  unsigned long long total = 0;
  int smax = 0;
  for (int row0 = blockIdx.x * MARK_WARPS; row0 < c; row0 += gridDim.x * MARK_WARPS) {
    const int row = row0 + warp;
    if (threadIdx.x < 2) s_cnt[threadIdx.x] = 0;
    __syncthreads();
    if (row < c) {
    unsigned long long rank = (none || all_ties || !tie_in_block) ? 0ull : rowbase[row];
    int s = 0;
    // a lane takes four consecutive columns (Bw % 8 == 0): one 16-byte load of the weights, one of
    // the norms and one 4-byte store of mask bytes per 128 columns
    for (int base = 0; base < Bw; base += 128) {
      const int jj = base + 4 * lane;
      const bool in = jj < Bw;
      float4 wv = make_float4(0.f, 0.f, 0.f, 0.f), xv = wv;
      if (in) {
        wv = *reinterpret_cast<const float4*>(Wc + (int64_t)row * b + j1 + jj);
        xv = __ldg(reinterpret_cast<const float4*>(xnorm + j1 + jj));
      }
      const unsigned key[4] = {metric_key(wv.x, xv.x), metric_key(wv.y, xv.y),
                               metric_key(wv.z, xv.z), metric_key(wv.w, xv.w)};
      bool pr[4];
      int ntie = 0;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        pr[e] = in && !none && key[e] < tau;
        ntie += (in && !none && key[e] == tau) ? 1 : 0;
      }
      if (__any_sync(0xffffffffu, ntie > 0)) {  // warp-uniform; rare outside tie-heavy blocks
        // ties in (row, column) order: ties of lower lanes come first, then this lane's in order
        int incl = ntie;
        for (int o = 1; o < 32; o <<= 1) {
          const int v = __shfl_up_sync(0xffffffffu, incl, o);
          if (lane >= o) incl += v;
        }
        unsigned long long myrank = rank + (unsigned long long)(incl - ntie);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          if (in && !none && key[e] == tau) {
            pr[e] = all_ties || myrank < need;
            ++myrank;
          }
        }
        rank += (unsigned long long)__shfl_sync(0xffffffffu, incl, 31);
      }
      if (in) {
        uchar4 mb;
        mb.x = pr[0] ? 1 : 0;
        mb.y = pr[1] ? 1 : 0;
        mb.z = pr[2] ? 1 : 0;
        mb.w = pr[3] ? 1 : 0;
        *reinterpret_cast<uchar4*>(mask + (int64_t)row * b + j1 + jj) = mb;
      }
      int cnt = (int)pr[0] + (int)pr[1] + (int)pr[2] + (int)pr[3];
      for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
      s += cnt;
    }
    total += s;
    smax = s > smax ? s : smax;
    if (lane == 0) {
      // rows that remove more than half of the block are solved in the complement form
      const int kind = (s > Bw - s) ? 1 : 0;
      s_rows[kind][atomicAdd(&s_cnt[kind], 1u)] = row;
    }
    }
    __syncthreads();
    if (threadIdx.x < 2 && s_cnt[threadIdx.x])
      s_base[threadIdx.x] = atomicAdd(&list_counts[threadIdx.x], s_cnt[threadIdx.x]);
    __syncthreads();
    if (threadIdx.x < MARK_WARPS) {
      if (threadIdx.x < s_cnt[0]) row_lists[s_base[0] + threadIdx.x] = s_rows[0][threadIdx.x];
      if (threadIdx.x < s_cnt[1]) row_lists[(size_t)c + s_base[1] + threadIdx.x] = s_rows[1][threadIdx.x];
    }
    __syncthreads();
  }
  // one update of the block's count and of the largest system per CTA
  if (threadIdx.x < 2) s_cnt[threadIdx.x] = 0;
  __syncthreads();
  if (lane == 0) {
    if (total) atomicAdd(&s_cnt[0], (unsigned)total);
    if (smax) atomicMax(&s_cnt[1], (unsigned)smax);
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    if (s_cnt[0]) atomicAdd(&st->blk_count, (unsigned long long)s_cnt[0]);
    if (s_cnt[1]) atomicMax(&stats->max_s, (int)s_cnt[1]);
  }
  // ---- the last CTA closes the block: budget, statistics, state of the next block's selection
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) s_last = (atomicAdd(&st->mark_ticket, 1u) == gridDim.x - 1) ? 1 : 0;
  __syncthreads();
  if (!s_last || threadIdx.x != 0) return;
  __threadfence();
  volatile SweepState* vs = st;
  const unsigned long long cnt = vs->blk_count;
  const long long r_new = vs->r - (long long)cnt;
  st->r = r_new;
  stats->r_left = r_new;
  if (!none) {
    stats->n_tied += (long long)(vs->count_eq - vs->need_eq);
    stats->last_threshold_bits = tau;
    st->tau_prev = tau;
  }
  if (r_ext) *r_ext = r_new;
  stats->n_pruned += (long long)cnt;
  stats->n_blocks += 1;
  st->blk_count = 0;
  st->mark_ticket = 0;
  // next block: bracket around this threshold when there is one, else a full radix select
  const unsigned half_window = 1u << ((vs->wide ? WINDOW_LOG2_WIDE : WINDOW_LOG2) - 1);
  const bool bracket = !none && tau >= half_window;
  st->have_prev = bracket ? 1 : 0;
  st->lo = bracket ? tau - half_window : 0u;
  st->prefix = 0;
  st->phase = bracket ? PH_BRACKET : PH_RADIX0;
}

// n:m: one thread per (row, group of m columns); the n smallest keys, lower column on ties.
__global__ void __launch_bounds__(256)
nm_mark_kernel(const float* __restrict__ Wc, const float* __restrict__ xnorm,
               uint8_t* __restrict__ mask, int c, int b, int j1, int Bw, int n, int m,
               thanos_stats_t* stats, const uint8_t* __restrict__ row_skip, int n_skip) {
  const int groups = Bw / m;
  int64_t idx = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (idx == 0) {  // launches of one sweep are ordered, so one thread can keep the books
    stats->n_pruned += (long long)(c - n_skip) * groups * n;
    stats->n_blocks += 1;
  }
  if (idx >= (int64_t)c * groups) return;
  int row = (int)(idx / groups), g = (int)(idx % groups);
  const float* w = Wc + (int64_t)row * b + j1 + g * m;
  const float* x = xnorm + j1 + g * m;
  unsigned key[32];
  for (int e = 0; e < m; ++e) key[e] = metric_key(w[e], __ldg(&x[e]));
  uint8_t* mo = mask + (int64_t)row * b + j1 + g * m;
  if (row_skip && row_skip[row]) {  // outlier row (Algorithm 4's row loop stops before them)
    for (int e = 0; e < m; ++e) mo[e] = 0;
    return;
  }
  for (int e = 0; e < m; ++e) {
    // rank of e = number of entries that come before it in (key, column) order
    int rk = 0;
    for (int f = 0; f < m; ++f) rk += (key[f] < key[e]) || (key[f] == key[e] && f < e);
    mo[e] = rk < n ? 1 : 0;
  }
}

__global__ void fold_tc_status_kernel(thanos_stats_t* stats, const int32_t* tc_status) {
  if (*tc_status != 0 && stats->status == 0) stats->status = *tc_status;
}

// ------------------------------------------------------------------ dtype conversion
__global__ void to_f32_kernel(const __nv_bfloat16* __restrict__ in, float* __restrict__ out,
                              int64_t n) {
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (; i < n; i += stride) out[i] = __bfloat162float(in[i]);
}

__global__ void to_bf16_kernel(const float* __restrict__ in, __nv_bfloat16* __restrict__ out,
                               int64_t n) {
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (; i < n; i += stride) out[i] = __float2bfloat16_rn(in[i]);
}

// A single block step that continues a sweep: `stats` still holds what the previous block step
// left (threshold of that block, whether a bracket has missed so far), so the selection starts
// from the same bracket the whole-layer sweep would use.  A zeroed `stats` leaves the state on the
// four radix passes.
__global__ void seed_select_kernel(SweepState* st, const thanos_stats_t* stats) {
  if (stats->n_blocks <= 0) return;
  const int wide = stats->select_misses > 0 ? 1 : 0;
  const unsigned tau = stats->last_threshold_bits;
  const unsigned half_window = 1u << ((wide ? WINDOW_LOG2_WIDE : WINDOW_LOG2) - 1);
  st->wide = wide;
  if (tau >= half_window) {
    st->tau_prev = tau;
    st->have_prev = 1;
    st->lo = tau - half_window;
    st->phase = PH_BRACKET;
  }
}

__global__ void init_sweep_kernel(SweepState* st, thanos_stats_t* stats, long long r) {
  SweepState z0 = {};
  z0.r = r;
  z0.phase = PH_RADIX0;
  *st = z0;
  thanos_stats_t z = {};
  z.r_left = r;
  *stats = z;
}

// ------------------------------------------------------------------ outlier rows (Algorithm 4)
// h_i = ||W_i X||^2 = 1/2 W_i H W_i^T from T = W H: one warp per row.
__global__ void __launch_bounds__(256)
row_loss_kernel(const float* __restrict__ Wc, const float* __restrict__ Tm, int c, int b,
                float* __restrict__ h) {
  const int lane = threadIdx.x & 31;
  const int row = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (row >= c) return;
  const float4* w = reinterpret_cast<const float4*>(Wc + (int64_t)row * b);
  const float4* t = reinterpret_cast<const float4*>(Tm + (int64_t)row * b);
  double acc = 0.0;
  for (int q = lane; q < (b >> 2); q += 32) {
    const float4 a = w[q], v = t[q];
    acc += (double)a.x * v.x + (double)a.y * v.y + (double)a.z * v.z + (double)a.w * v.w;
  }
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if (lane == 0) h[row] = fmaxf((float)(0.5 * acc), 0.f);
}

// The n_out rows with the largest h (order (h, row): of equal losses the higher row index is the
// larger) get flag 1.  One CTA: radix select of the n_out-th largest key, then the ties.
__global__ void __launch_bounds__(1024)
outlier_rows_kernel(const float* __restrict__ h, int c, int n_out, uint8_t* __restrict__ flags) {
  __shared__ unsigned hist[256];
  __shared__ unsigned s_prefix, s_k, s_gt;
  const int tid = threadIdx.x;
  if (tid == 0) {
    s_prefix = 0;
    s_k = (unsigned)n_out;  // rank from the top still to resolve
  }
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    if (tid < 256) hist[tid] = 0;
    __syncthreads();
    const unsigned prefix = s_prefix;
    for (int i = tid; i < c; i += 1024) {
      const unsigned key = __float_as_uint(h[i]);
      if (pass == 0 || (key >> (shift + 8)) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (tid == 0) {
      unsigned k = s_k, bin = 255;
      for (;; --bin) {  // from the largest digit down
        if (hist[bin] >= k || bin == 0) break;
        k -= hist[bin];
      }
      s_prefix = (prefix << 8) | bin;
      s_k = k;
    }
    __syncthreads();
  }
  const unsigned tau = s_prefix;  // key of the n_out-th largest loss
  if (tid == 0) s_gt = 0;
  __syncthreads();
  unsigned gt = 0;
  for (int i = tid; i < c; i += 1024) {
    const unsigned key = __float_as_uint(h[i]);
    flags[i] = key > tau ? 1 : 0;
    gt += key > tau;
  }
  atomicAdd(&s_gt, gt);
  __syncthreads();
  if (tid == 0) {
    int need = n_out - (int)s_gt;
    for (int i = c - 1; i >= 0 && need > 0; --i) {
      if (__float_as_uint(h[i]) == tau) {
        flags[i] = 1;
        --need;
      }
    }
  }
}

struct SweepWs {
  float* Wc;   // fp32 working copy when the I/O dtype is not fp32
  __nv_bfloat16* D;    // [3][c, g B] change of the current block(s) (delta) as bf16 planes
  float* Ubb;  // [blocks, B, B] per-block matrices
  float* Vbb;
  float* G;
  float* S;
  __nv_bfloat16* P2;   // [3][b, b] bf16 planes; rows j1..j2 hold V_bb U[j1:j2, j2:] (columns >= j2)
  int32_t* tc_status;  // device status word of the tensor-core products
  unsigned* hist;
  SweepState* st;
  unsigned* rowcnt;
  unsigned long long* rowbase;
  unsigned* cand;         // keys copied out of the bracket window
  size_t cand_cap;
  int* row_lists;         // [2, c] rows of the current block by kind of system
  unsigned* list_counts;  // [2]
};

// n:m mode: blocks per group whose far update is applied once per group (the update of a block
// only has to reach the group's own columns before the next block is masked, because the n:m
// mask reads nothing but its block).  Groups span 512 columns; small layers gain nothing.
int lazy_group(int64_t b, int B) {
  if (b < 2048 || B >= 512) return 1;
  const int g = 512 / B;
  return g < 1 ? 1 : (g > 8 ? 8 : g);
}

// room for one key in eight of the layer (the bracket window holds about one in 130)
size_t cand_capacity(int64_t c, int64_t b) {
  size_t n = (size_t)c * (size_t)b / 8;
  if (n < 4096) n = 4096;
  if (n > ((size_t)1 << 31)) n = (size_t)1 << 31;
  return n;
}

bool carve(SweepWs& w, void* workspace, size_t ws_bytes, int64_t c, int64_t b, int32_t B,
           bool need_wc) {
  Arena ar(workspace, ws_bytes);
  const size_t blocks = (size_t)ceil_div(b, B);
  w.Wc = need_wc ? ar.take<float>((size_t)c * b) : nullptr;
  w.D = ar.take<__nv_bfloat16>(3 * (size_t)c * B * lazy_group(b, B));
  w.Ubb = ar.take<float>(blocks * B * B);
  w.Vbb = ar.take<float>(blocks * B * B);
  w.G = ar.take<float>(blocks * B * B);
  w.S = ar.take<float>(blocks * B * B);
  w.P2 = ar.take<__nv_bfloat16>(3 * (size_t)b * b);
  w.tc_status = ar.take<int32_t>(4);
  w.hist = ar.take<unsigned>(HIST_BINS);
  w.st = ar.take<SweepState>(1);
  w.rowcnt = ar.take<unsigned>((size_t)c);
  w.rowbase = ar.take<unsigned long long>((size_t)c);
  w.cand_cap = cand_capacity(c, b);
  w.cand = ar.take<unsigned>(w.cand_cap);
  w.row_lists = ar.take<int>(2 * (size_t)c);
  w.list_counts = ar.take<unsigned>(2);
  return ar.ok();
}

// G, S, V_bb of every block and P2, once per sweep.
thanos_status_t prepare_blocks(const float* U, int b, int B, const SweepWs& w,
                               cudaStream_t stream) {
  const int blocks = (int)ceil_div(b, B);
  {
    static std::atomic<unsigned long long> done{0};
    THANOS_CUDA(ensure_max_dyn_smem(block_inverse_kernel, (int)block_inverse_smem(512), done));
  }
  block_inverse_kernel<<<dim3((unsigned)ceil_div(B, INV_STRIP), (unsigned)blocks), 256,
                         block_inverse_smem(B), stream>>>(U, w.Ubb, w.Vbb, b, B);
  THANOS_CHECK_LAUNCH();
  dim3 gg((unsigned)ceil_div(B, 64), (unsigned)ceil_div(B, 64), (unsigned)blocks);
  block_gram_kernel<0><<<gg, 256, 0, stream>>>(w.Ubb, w.G, b, B);
  THANOS_CHECK_LAUNCH();
  block_gram_kernel<1><<<gg, 256, 0, stream>>>(w.Vbb, w.S, b, B);
  THANOS_CHECK_LAUNCH();
  if (b > B) {
    dim3 gp((unsigned)ceil_div(b - B, 64), (unsigned)ceil_div(B, 64), (unsigned)blocks);
    block_rows_kernel<<<gp, 256, 0, stream>>>(U, w.Vbb, w.P2, b, B);
    THANOS_CHECK_LAUNCH();
  }
  return THANOS_OK;
}

thanos_status_t block_step(float* Wc, uint8_t* mask, int c, int b, const float* xnorm,
                           thanos_mode_t mode, int n, int m, int B, int j1, int64_t* r_ext,
                           const SweepWs& w, thanos_stats_t* stats, cudaStream_t stream,
                           const uint8_t* row_skip = nullptr, int n_skip = 0, int d_col = 0,
                           int ldd = 0, int upd_end = -1) {
  // delta goes to columns [d_col, d_col + Bw) of the plane buffer (leading dimension ldd); the
  // update is applied to columns [j2, upd_end) of W
  const int Bw = (b - j1 < B) ? b - j1 : B;
  const int j2 = j1 + Bw;
  const int bb = j1 / B;
  if (ldd == 0) ldd = B;
  if (upd_end < 0) upd_end = b;
  int s_fixed = -1;
  if (mode == THANOS_UNSTRUCTURED) {
    // bracket + refine, or the four radix passes, or bracket + four radix passes when it misses
    const int sg = c < NUM_SMS * 4 ? c : NUM_SMS * 4;
    // residuals beyond the L2 stream from HBM and want more loads in flight
    const bool big = (size_t)c * (size_t)(b - j1) * sizeof(float) > ((size_t)96 << 20);
    const int sg2 = sg < NUM_SMS * 2 ? sg : NUM_SMS * 2;
    // the pass over the residual (bracket, or the first radix pass)
    if (big)
      select_pass_kernel<4><<<sg, 256, 0, stream>>>(Wc, xnorm, c, b, j1, w.st, w.hist, r_ext,
                                                    w.list_counts, 1, stats, w.cand,
                                                    (unsigned)w.cand_cap);
    else
      select_pass_kernel<2><<<sg, 256, 0, stream>>>(Wc, xnorm, c, b, j1, w.st, w.hist, r_ext,
                                                    w.list_counts, 1, stats, w.cand,
                                                    (unsigned)w.cand_cap);
    THANOS_CHECK_LAUNCH();
    {
      // everything else behind grid barriers in one launch (sg2 <= 2 CTAs per SM: co-resident):
      // the refine pass over the copied keys, or what is left of a radix route, then the ties
      const float* a_Wc = Wc;
      const float* a_xn = xnorm;
      int a_c = c, a_b = b, a_j1 = j1, a_bw = Bw;
      SweepState* a_st = w.st;
      unsigned* a_hist = w.hist;
      unsigned* a_lc = w.list_counts;
      thanos_stats_t* a_stats = stats;
      unsigned* a_cand = w.cand;
      unsigned a_cap = (unsigned)w.cand_cap;
      unsigned* a_rowcnt = w.rowcnt;
      unsigned long long* a_rowbase = w.rowbase;
      void* args[] = {&a_Wc, &a_xn, &a_c, &a_b, &a_j1, &a_bw, &a_st, &a_hist, &a_lc, &a_stats, &a_cand,
                      &a_cap, &a_rowcnt, &a_rowbase};
      const void* fn = big ? reinterpret_cast<const void*>(&select_rest_kernel<4>)
                           : reinterpret_cast<const void*>(&select_rest_kernel<2>);
      if (cudaLaunchCooperativeKernel(fn, dim3((unsigned)sg2), dim3(256), args, 0, stream) !=
          cudaSuccess)
        return THANOS_ERR_CUDA;
      count_launch();
    }
    int mg = (int)ceil_div(c, MARK_WARPS);
    if (mg > NUM_SMS * 2) mg = NUM_SMS * 2;
    mark_block_kernel<<<mg, 32 * MARK_WARPS, 0, stream>>>(Wc, xnorm, mask, c, b, j1, Bw, w.st, w.rowbase,
                                              w.row_lists, w.list_counts, stats, r_ext);
    THANOS_CHECK_LAUNCH();
  } else {
    s_fixed = Bw / m * n;
    int64_t items = (int64_t)c * (Bw / m);
    nm_mark_kernel<<<(unsigned)ceil_div(items, 256), 256, 0, stream>>>(Wc, xnorm, mask, c, b, j1,
                                                                      Bw, n, m, stats, row_skip, n_skip);
    THANOS_CHECK_LAUNCH();
  }
  THANOS_TRY(launch_block_solve(Wc, mask, w.G + (size_t)bb * B * B, w.S + (size_t)bb * B * B, B,
                                w.D + d_col, (int64_t)c * ldd, c, b, j1, Bw, ldd, s_fixed,
                                w.row_lists, w.list_counts, stats, stream));
  if (j2 < upd_end) {
    // W[:, j2:upd_end] += delta P2[j1:j2, j2:upd_end]
    TcGemmArgs g;
    g.D = Wc + j2;
    g.ldd = b;
    g.A = w.D + d_col;
    g.lda = ldd;
    g.a_plane = (int64_t)c * ldd;
    g.B = w.P2 + (int64_t)j1 * b + j2;
    g.ldb = b;
    g.b_plane = (int64_t)b * b;
    g.b_kmajor = 0;
    g.M = c;
    g.N = upd_end - j2;
    g.K = Bw;
    g.alpha = 1.f;
    g.accumulate = 1;
    g.status = w.tc_status;
    THANOS_TRY(tc_gemm_split3(g, stream));
  }
  return THANOS_OK;
}

}  // namespace

// dtype conversion of a whole weight matrix (bf16 I/O <-> fp32 working copy)
thanos_status_t convert_to_f32(const __nv_bfloat16* in, float* out, int64_t n, cudaStream_t stream) {
  to_f32_kernel<<<NUM_SMS * 8, 256, 0, stream>>>(in, out, n);
  THANOS_CHECK_LAUNCH();
  return THANOS_OK;
}

thanos_status_t convert_to_bf16(const float* in, __nv_bfloat16* out, int64_t n, cudaStream_t stream) {
  to_bf16_kernel<<<NUM_SMS * 8, 256, 0, stream>>>(in, out, n);
  THANOS_CHECK_LAUNCH();
  return THANOS_OK;
}

size_t prune_workspace_bytes(int64_t c, int64_t b, int32_t B, thanos_dtype_t dtype) {
  size_t t = 0;
  const size_t blocks = (size_t)ceil_div(b, B);
  if (dtype != THANOS_F32) t += round_up((size_t)c * b * sizeof(float), 256);
  t += round_up(3 * (size_t)c * B * lazy_group(b, B) * sizeof(__nv_bfloat16), 256);
  t += 4 * round_up(blocks * B * B * sizeof(float), 256);
  t += round_up(3 * (size_t)b * b * sizeof(__nv_bfloat16), 256) + 256;
  t += round_up(HIST_BINS * sizeof(unsigned), 256);
  t += round_up(sizeof(SweepState), 256);
  t += round_up((size_t)c * sizeof(unsigned), 256);
  t += round_up((size_t)c * sizeof(unsigned long long), 256);
  t += round_up(2 * (size_t)c * sizeof(int), 256);
  t += round_up(cand_capacity(c, b) * sizeof(unsigned), 256);
  t += 256;
  return t + 256;
}

thanos_status_t validate_sweep_args(int64_t c, int64_t b, thanos_mode_t mode, double p, int32_t n,
                                    int32_t m, int32_t B) {
  if (c < 1 || b < 1 || c > (1 << 30) || b > (1 << 30)) return THANOS_ERR_SHAPE;
  if (b % 8 != 0 || B < 1 || B > 512 || B % 8 != 0) return THANOS_ERR_SHAPE;
  if (mode == THANOS_UNSTRUCTURED) {
    if (!(p >= 0.0 && p < 1.0)) return THANOS_ERR_INVALID_ARG;
    if (!solve_supported(B, B / 2)) return THANOS_ERR_SHAPE;
  } else if (mode == THANOS_NM) {
    if (!(n > 0 && n < m && m <= 32)) return THANOS_ERR_INVALID_ARG;
    if (B % m != 0 || b % m != 0) return THANOS_ERR_SHAPE;
    const int s = B / m * n;
    if (!solve_supported(s, s < B - s ? s : B - s)) return THANOS_ERR_SHAPE;
  } else {
    return THANOS_ERR_INVALID_ARG;
  }
  return THANOS_OK;
}

thanos_status_t prune_block_impl(float* Wc, uint8_t* mask, int64_t c, int64_t b, const float* U,
                                 const float* xnorm, thanos_mode_t mode, int32_t n, int32_t m,
                                 int32_t B, int64_t j1, int64_t* r_dev, void* workspace,
                                 size_t ws_bytes, thanos_stats_t* stats, cudaStream_t stream) {
  SweepWs w;
  if (!carve(w, workspace, ws_bytes, c, b, B, false)) return THANOS_ERR_WORKSPACE;
  THANOS_CUDA(cudaMemsetAsync(w.hist, 0, HIST_BINS * sizeof(unsigned), stream));
  THANOS_CUDA(cudaMemsetAsync(w.st, 0, sizeof(SweepState), stream));
  THANOS_CUDA(cudaMemsetAsync(w.tc_status, 0, 16, stream));
  if (mode == THANOS_UNSTRUCTURED) {
    seed_select_kernel<<<1, 1, 0, stream>>>(w.st, stats);
    THANOS_CHECK_LAUNCH();
  }
  THANOS_TRY(prepare_blocks(U, (int)b, B, w, stream));
  THANOS_TRY(block_step(Wc, mask, (int)c, (int)b, xnorm, mode, n, m, B, (int)j1, r_dev, w, stats,
                        stream));
  fold_tc_status_kernel<<<1, 1, 0, stream>>>(stats, w.tc_status);
  THANOS_CHECK_LAUNCH();
  return THANOS_OK;
}

namespace {

struct OutlierWs {
  __nv_bfloat16* Wp;  // [3][c, b] planes of the weights
  __nv_bfloat16* Hp;  // [3][b, b] planes of the Hessian
  float* T;           // [c, b] W H
  float* h;           // [c] row losses
  uint8_t* flags;     // [c] 1 = outlier row
};

}  // namespace

size_t outlier_extra_bytes(int64_t c, int64_t b) {
  size_t t = round_up(3 * (size_t)c * b * sizeof(__nv_bfloat16), 256);
  t += round_up(3 * (size_t)b * b * sizeof(__nv_bfloat16), 256);
  t += round_up((size_t)c * b * sizeof(float), 256);
  t += round_up((size_t)c * sizeof(float), 256);
  t += round_up((size_t)c, 256);
  return t + 256;
}

// Outlier rows (Algorithms 2 and 4): h = 1/2 rowdot(W, W H), then flag 1 on the n_out rows with
// the largest h.  scratch holds outlier_extra_bytes(c, b); *flags_dev points into it.
thanos_status_t outlier_row_flags(const float* Wc, const float* H, int64_t c, int64_t b, int n_out,
                                  void* scratch, size_t scratch_bytes, uint8_t** flags_dev,
                                  int32_t* tc_status, cudaStream_t stream) {
  const int64_t nel = c * b;
  Arena ar(scratch, scratch_bytes);
  OutlierWs o;
  o.Wp = ar.take<__nv_bfloat16>(3 * (size_t)nel);
  o.Hp = ar.take<__nv_bfloat16>(3 * (size_t)b * b);
  o.T = ar.take<float>((size_t)nel);
  o.h = ar.take<float>((size_t)c);
  o.flags = ar.take<uint8_t>((size_t)c);
  if (!ar.ok()) return THANOS_ERR_WORKSPACE;
  THANOS_TRY(split3_planes(Wc, b, c, b, o.Wp, b, nel, stream));
  THANOS_TRY(split3_planes(H, b, b, b, o.Hp, b, b * b, stream));
  TcGemmArgs g;
  g.D = o.T;
  g.ldd = b;
  g.A = o.Wp;
  g.lda = b;
  g.a_plane = nel;
  g.B = o.Hp;
  g.ldb = b;
  g.b_plane = b * b;
  g.b_kmajor = 0;
  g.M = (int)c;
  g.N = (int)b;
  g.K = (int)b;
  g.status = tc_status;
  THANOS_TRY(tc_gemm_split3(g, stream));
  row_loss_kernel<<<(unsigned)ceil_div(c, 8), 256, 0, stream>>>(Wc, o.T, (int)c, (int)b, o.h);
  THANOS_CHECK_LAUNCH();
  outlier_rows_kernel<<<1, 1024, 0, stream>>>(o.h, (int)c, n_out, o.flags);
  THANOS_CHECK_LAUNCH();
  *flags_dev = o.flags;
  return THANOS_OK;
}

namespace {

// The whole sweep.  With H and alpha > 0 (n:m mode) the ceil(alpha c) rows with the largest
// h_i = 1/2 W_i H W_i^T are found first and left untouched (Algorithm 4, outlier rows).
thanos_status_t prune_layer_core(const void* W_in, void* W_out, uint8_t* mask_out,
                                 thanos_dtype_t wdtype, int64_t c, int64_t b, const float* U,
                                 const float* xnorm, thanos_mode_t mode, double p, int32_t n,
                                 int32_t m, int32_t B, void* workspace, size_t ws_bytes,
                                 thanos_stats_t* stats, cudaStream_t stream, const float* H,
                                 double alpha, uint8_t* row_flags_out) {
  SweepWs w;
  const bool need_wc = wdtype != THANOS_F32;
  if (!carve(w, workspace, ws_bytes, c, b, B, need_wc)) return THANOS_ERR_WORKSPACE;
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
  THANOS_CUDA(cudaMemsetAsync(w.hist, 0, HIST_BINS * sizeof(unsigned), stream));
  THANOS_CUDA(cudaMemsetAsync(w.tc_status, 0, 16, stream));
  const uint8_t* row_skip = nullptr;
  int n_skip = 0;
  if (H != nullptr) {
    // outlier rows: h = 1/2 rowdot(W, W H), then the ceil(alpha c) largest
    n_skip = alpha > 0.0 ? (int)ceil(alpha * (double)c - 1e-12) : 0;
    const size_t base = prune_workspace_bytes(c, b, B, wdtype);
    if (ws_bytes < base + outlier_extra_bytes(c, b)) return THANOS_ERR_WORKSPACE;
    uint8_t* flags = nullptr;
    THANOS_TRY(outlier_row_flags(Wc, H, c, b, n_skip, static_cast<char*>(workspace) + base,
                                 ws_bytes - base, &flags, w.tc_status, stream));
    if (row_flags_out)
      THANOS_CUDA(cudaMemcpyAsync(row_flags_out, flags, (size_t)c, cudaMemcpyDeviceToDevice,
                                  stream));
    row_skip = flags;
  }
  long long r = 0;
  if (mode == THANOS_UNSTRUCTURED) r = (long long)floor(p * (double)c * (double)b);
  init_sweep_kernel<<<1, 1, 0, stream>>>(w.st, stats, r);
  THANOS_CHECK_LAUNCH();
  THANOS_TRY(prepare_blocks(U, (int)b, B, w, stream));
  const int grp = mode == THANOS_NM ? lazy_group(b, B) : 1;
  if (grp == 1) {
    for (int64_t j1 = 0; j1 < b; j1 += B) {
      THANOS_TRY(block_step(Wc, mask_out, (int)c, (int)b, xnorm, mode, n, m, B, (int)j1, nullptr,
                            w, stats, stream, row_skip, n_skip));
    }
  } else {
    // n:m: the blocks of a group update the group's columns at once and everything to the right
    // of the group by one product over the whole group (K = grp B), which reads and writes
    // those weights once per group instead of once per block
    const int ldd = grp * B;
    for (int64_t g0 = 0; g0 < b; g0 += ldd) {
      const int64_t g_end = g0 + ldd < b ? g0 + ldd : b;
      for (int64_t j1 = g0; j1 < g_end; j1 += B) {
        THANOS_TRY(block_step(Wc, mask_out, (int)c, (int)b, xnorm, mode, n, m, B, (int)j1, nullptr,
                              w, stats, stream, row_skip, n_skip, (int)(j1 - g0), ldd,
                              (int)g_end));
      }
      if (g_end < b) {
        TcGemmArgs g;
        g.D = Wc + g_end;
        g.ldd = b;
        g.A = w.D;
        g.lda = ldd;
        g.a_plane = c * ldd;
        g.B = w.P2 + g0 * b + g_end;
        g.ldb = b;
        g.b_plane = b * b;
        g.b_kmajor = 0;
        g.M = (int)c;
        g.N = (int)(b - g_end);
        g.K = (int)(g_end - g0);
        g.alpha = 1.f;
        g.accumulate = 1;
        g.status = w.tc_status;
        THANOS_TRY(tc_gemm_split3(g, stream));
      }
    }
  }
  fold_tc_status_kernel<<<1, 1, 0, stream>>>(stats, w.tc_status);
  THANOS_CHECK_LAUNCH();
  if (need_wc) {
    THANOS_TRY(convert_to_bf16(Wc, static_cast<__nv_bfloat16*>(W_out), nel, stream));
  }
  return THANOS_OK;
}

}  // namespace

thanos_status_t prune_layer_impl(const void* W_in, void* W_out, uint8_t* mask_out,
                                 thanos_dtype_t wdtype, int64_t c, int64_t b, const float* U,
                                 const float* xnorm, thanos_mode_t mode, double p, int32_t n,
                                 int32_t m, int32_t B, void* workspace, size_t ws_bytes,
                                 thanos_stats_t* stats, cudaStream_t stream) {
  return prune_layer_core(W_in, W_out, mask_out, wdtype, c, b, U, xnorm, mode, p, n, m, B,
                          workspace, ws_bytes, stats, stream, nullptr, 0.0, nullptr);
}

size_t prune_outliers_workspace_bytes(int64_t c, int64_t b, int32_t B, thanos_dtype_t dtype) {
  return prune_workspace_bytes(c, b, B, dtype) + outlier_extra_bytes(c, b);
}

thanos_status_t prune_layer_outliers_impl(const void* W_in, void* W_out, uint8_t* mask_out,
                                          thanos_dtype_t wdtype, int64_t c, int64_t b,
                                          const float* U, const float* xnorm, const float* H,
                                          int32_t n, int32_t m, int32_t B, double alpha,
                                          uint8_t* row_flags_out, void* workspace, size_t ws_bytes,
                                          thanos_stats_t* stats, cudaStream_t stream) {
  return prune_layer_core(W_in, W_out, mask_out, wdtype, c, b, U, xnorm, THANOS_NM, 0.0, n, m, B,
                          workspace, ws_bytes, stats, stream, H, alpha, row_flags_out);
}

}  // namespace thanos
