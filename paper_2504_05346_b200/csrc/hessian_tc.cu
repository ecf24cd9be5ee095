// H += 2 X^T X on the 5th-generation tensor cores (Section 3.2: H = 2 X X^T, paper's X = X^T here).
//
// One CTA per SM, persistent over work units (output tile x token slice).  Roles:
//   warp 0      TMA producer: 64-token x 64-feature boxes of X into a 4-stage shared-memory ring
//   warp 1      tcgen05.mma issuer: 128 x 256 x 16 bf16 MMAs, both operands MN-major (the
//               contraction runs over tokens, which is the strided dimension of X)
//   warps 2..9  accumulation: every 512 tokens the TMEM accumulator is drained into fp32
//               registers (round-to-nearest adds), so no TMEM sum runs longer than 32 MMAs;
//               at the end of a unit 2*acc is added to H[i, j] and to the mirror H[j, i].
// TMEM: two 128 x 256 fp32 accumulators (all 512 columns), so draining overlaps the next MMAs.
// Only tiles that touch the upper triangle are computed.  fp32 inputs are first split into
// three bf16 planes (x = h + m + l); a stage then holds all three planes of 32 tokens, and the six
// significant plane products hh, hm, mh, hl, lh, mm are issued from it.
//
// Every wait is bounded: on expiry the CTA raises an abort flag, records THANOS_ERR_TIMEOUT in
// the status word, drains, frees its TMEM and returns.
#include "tc_common.cuh"

namespace thanos {

namespace {

constexpr int TM = 128;           // tile rows (features i)
constexpr int TN = 256;           // tile columns (features j)
constexpr int NTHREADS = 320;

// Pipeline geometry.  One plane (bf16 input): 64 tokens per stage, 4 boxes of 64 features for the j
// block and 2 for the i block (48 KB), four stages, the accumulator drained every 8 stages = 512
// tokens = 32 MMAs.  Three planes (split fp32 input): all three planes of both blocks for 32
// tokens per stage (72 KB, three stages), from which the six plane products are issued -- every
// plane is loaded once per token step, not once per product --, drained every 3 stages = 96
// tokens = 36 MMAs.
template <bool P3>
struct Geo {
  static constexpr int BK = P3 ? 32 : 64;
  static constexpr int STAGES = P3 ? 3 : 4;
  static constexpr int FLUSH_STAGES = P3 ? 3 : 8;
  static constexpr int BOX_BYTES = 64 * BK * 2;            // one 64-feature x BK-token bf16 box
  static constexpr int PLANE_BYTES = 6 * BOX_BYTES;        // 4 boxes of the j block, 2 of the i block
  static constexpr int A_OFFSET = 4 * BOX_BYTES;
  static constexpr int STAGE_BYTES = (P3 ? 3 : 1) * PLANE_BYTES;
  static constexpr size_t SMEM_BYTES = (size_t)STAGES * STAGE_BYTES + 1024 /*align*/ + 256 /*barriers*/;
};

struct Params {
  float* H;
  int32_t* status;
  int b;
  int n_tok;
  int nI, nJ;          // 128-row blocks, 256-column blocks
  int n_tiles;
  int n_slices;
  int slice_tokens;    // multiple of BK
  int n_combo;         // 1 (bf16 input) or 6 (split fp32 input)
  int plane_a[6];
  int plane_b[6];
};

using namespace tc;

// Shared-memory matrix descriptor for an MN-major bf16 operand stored as 64-feature x 64-token
// boxes with the 128-byte swizzle: a token is one 128-byte row, 8 tokens form a 1024-byte
// swizzle atom (stride offset), the next 64 features live one box further (leading offset).
__device__ __forceinline__ uint64_t make_desc(uint32_t smem_addr, uint32_t box_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)(box_bytes >> 4) << 16;            // leading-dimension byte offset
  d |= (uint64_t)(1024u >> 4) << 32;                // stride-dimension byte offset
  d |= (uint64_t)1 << 46;                           // descriptor version for sm_100
  d |= (uint64_t)2 << 61;                           // 128-byte swizzle
  return d;
}

// kind::f16 instruction descriptor: D fp32, A and B bf16, both MN-major, M = 128, N = 256.
__device__ __forceinline__ uint32_t make_idesc() {
  uint32_t d = 0;
  d |= 1u << 4;                  // D format: f32
  d |= 1u << 7;                  // A format: bf16
  d |= 1u << 10;                 // B format: bf16
  d |= 1u << 15;                 // A is MN-major
  d |= 1u << 16;                 // B is MN-major
  d |= (uint32_t)(TN >> 3) << 17;
  d |= (uint32_t)(TM >> 4) << 24;
  return d;
}

struct Unit {
  int I, J, t0, nst;
  bool diag;
};

__device__ __forceinline__ Unit decode_unit(const Params& p, int u, int bk) {
  Unit r;
  int tile = u % p.n_tiles;
  int slice = u / p.n_tiles;
  int J = 0;
  for (;;) {
    int cnt = 2 * J + 2 < p.nI ? 2 * J + 2 : p.nI;
    if (tile < cnt) break;
    tile -= cnt;
    ++J;
  }
  r.I = tile;
  r.J = J;
  r.diag = (tile >> 1) == J;
  r.t0 = slice * p.slice_tokens;
  int t1 = r.t0 + p.slice_tokens;
  if (t1 > p.n_tok) t1 = p.n_tok;
  r.nst = (t1 - r.t0 + bk - 1) / bk;
  if (r.nst < 0) r.nst = 0;
  return r;
}

template <bool P3>
__global__ void __launch_bounds__(NTHREADS, 1)
hessian_tc_kernel(const __grid_constant__ CUtensorMap tmap, const Params p) {
  using G = Geo<P3>;
  constexpr int BK = G::BK, STAGES = G::STAGES, FLUSH_STAGES = G::FLUSH_STAGES;
  constexpr int BOX_BYTES = G::BOX_BYTES, STAGE_BYTES = G::STAGE_BYTES, A_OFFSET = G::A_OFFSET;
  constexpr int PLANE_BYTES = G::PLANE_BYTES;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)STAGES * STAGE_BYTES);
  // bars[0..3] full, [4..7] empty, [8..9] tmem full, [10..11] tmem empty (STAGES <= 4)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 12);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 13);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t bar_base = smem_u32(bars);
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (4 + s); };
  auto tfull_bar = [&](int q) { return bar_base + 8u * (8 + q); };
  auto tempty_bar = [&](int q) { return bar_base + 8u * (10 + q); };

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int q = 0; q < 2; ++q) {
      mbar_init(tfull_bar(q), 1);
      mbar_init(tempty_bar(q), 8);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(tmem_slot)),
                 "r"(512)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int n_units = p.n_tiles * p.n_slices;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    int s = 0;
    uint32_t phase = 0;
    bool ok = true;
    for (int u = blockIdx.x; u < n_units && ok; u += gridDim.x) {
      const Unit un = decode_unit(p, u, BK);
      const int total = P3 ? un.nst : un.nst * p.n_combo;
      for (int kk = 0; kk < total && ok; ++kk) {
        const int combo = P3 ? 0 : kk / un.nst;
        const int ks = kk - combo * un.nst;
        const int pa = p.plane_a[combo], pb = p.plane_b[combo];
        // on a diagonal tile the i block is one half of the j block (of the same plane)
        const bool shortcut = un.diag && (P3 || pa == pb);
        ok = mbar_wait(empty_bar(s), phase ^ 1u, abort_flag);
        if (ok && lane == 0) {
          const uint32_t dst = smem_base + (uint32_t)s * STAGE_BYTES;
          const int y = un.t0 + ks * BK;
          mbar_expect_tx(full_bar(s), (P3 ? 3 : 1) * (shortcut ? 4 * BOX_BYTES : 6 * BOX_BYTES));
#pragma unroll
          for (int pl = 0; pl < (P3 ? 3 : 1); ++pl) {
            const uint32_t d0 = dst + (uint32_t)pl * PLANE_BYTES;
#pragma unroll
            for (int i = 0; i < 4; ++i)
              tma_load_3d(d0 + i * BOX_BYTES, &tmap, full_bar(s), un.J * TN + 64 * i, y, P3 ? pl : pb);
            if (!shortcut) {
#pragma unroll
              for (int i = 0; i < 2; ++i)
                tma_load_3d(d0 + A_OFFSET + i * BOX_BYTES, &tmap, full_bar(s), un.I * TM + 64 * i, y,
                            P3 ? pl : pa);
            }
          }
        }
        __syncwarp();
        if (++s == STAGES) {
          s = 0;
          phase ^= 1u;
        }
      }
    }
    // let copies that are still in flight land before the CTA's shared memory goes away
    if (!ok) {
      for (int i = 0; i < 2000; ++i) __nanosleep(1000);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    const uint32_t idesc = make_idesc();
    int s = 0, q = 0;
    uint32_t phase = 0, tphase = 0;
    bool ok = true;
    for (int u = blockIdx.x; u < n_units && ok; u += gridDim.x) {
      const Unit un = decode_unit(p, u, BK);
      const int total = P3 ? un.nst : un.nst * p.n_combo;
      for (int g0 = 0; g0 < total && ok; g0 += FLUSH_STAGES) {
        const int g1 = g0 + FLUSH_STAGES < total ? g0 + FLUSH_STAGES : total;
        ok = mbar_wait(tempty_bar(q), tphase ^ 1u, abort_flag);
        tc_fence_after();
        for (int kk = g0; kk < g1 && ok; ++kk) {
          const int combo = P3 ? 0 : kk / un.nst;
          ok = mbar_wait(full_bar(s), phase, abort_flag);
          tc_fence_after();
          if (ok && lane == 0) {
            const uint32_t stage = smem_base + (uint32_t)s * STAGE_BYTES;
#pragma unroll
            for (int cb = 0; cb < (P3 ? 6 : 1); ++cb) {
              const int pa = p.plane_a[P3 ? cb : combo], pb = p.plane_b[P3 ? cb : combo];
              const bool shortcut = un.diag && (P3 || pa == pb);
              const uint32_t sb = stage + (P3 ? (uint32_t)pb * PLANE_BYTES : 0u);
              const uint32_t pa_base = stage + (P3 ? (uint32_t)pa * PLANE_BYTES : 0u);
              const uint32_t sa =
                  shortcut ? pa_base + (uint32_t)(un.I & 1) * 2 * BOX_BYTES : pa_base + A_OFFSET;
#pragma unroll
              for (int k4 = 0; k4 < BK / 16; ++k4) {
                const uint64_t adesc = make_desc(sa + k4 * 2048, BOX_BYTES);
                const uint64_t bdesc = make_desc(sb + k4 * 2048, BOX_BYTES);
                tc_mma_bf16(tmem_base + (uint32_t)q * TN, adesc, bdesc, idesc,
                            (kk > g0 || cb > 0 || k4 > 0) ? 1u : 0u);
              }
            }
            tc_commit(empty_bar(s));
          }
          __syncwarp();
          if (++s == STAGES) {
            s = 0;
            phase ^= 1u;
          }
        }
        if (ok && lane == 0) tc_commit(tfull_bar(q));
        __syncwarp();
        if (++q == 2) {
          q = 0;
          tphase ^= 1u;
        }
      }
    }
  } else {
    // ------------------------------------------------------------ accumulate + write out
    const int ew = warp - 2;
    const int g = warp & 3;     // TMEM lane quarter this warp may read
    const int h = ew >> 2;      // column half
    int q = 0;
    uint32_t tphase = 0;
    bool ok = true;
    for (int u = blockIdx.x; u < n_units && ok; u += gridDim.x) {
      const Unit un = decode_unit(p, u, BK);
      const int total = P3 ? un.nst : un.nst * p.n_combo;
      float acc[128];
#pragma unroll
      for (int k = 0; k < 128; ++k) acc[k] = 0.f;
      for (int g0 = 0; g0 < total && ok; g0 += FLUSH_STAGES) {
        ok = mbar_wait(tfull_bar(q), tphase, abort_flag);
        tc_fence_after();
        if (ok) {
          const uint32_t taddr = tmem_base + ((uint32_t)(32 * g) << 16) + (uint32_t)q * TN + h * 128;
#pragma unroll
          for (int cc = 0; cc < 4; ++cc) {
            uint32_t v[32];
            tc_ld32(taddr + cc * 32, v);
            tc_wait_ld();
#pragma unroll
            for (int k = 0; k < 32; ++k) acc[cc * 32 + k] += __uint_as_float(v[k]);
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(tempty_bar(q));
        if (++q == 2) {
          q = 0;
          tphase ^= 1u;
        }
      }
      if (!ok || total == 0) continue;
      const int i = un.I * TM + 32 * g + lane;
      const int jbase = un.J * TN + h * 128;
      float* __restrict__ H = p.H;
      const int b = p.b;
      if (i < b) {
#pragma unroll
        for (int k = 0; k < 128; k += 4) {
          const int j = jbase + k;
          if (j + 3 < b && i < j) {
            red_add4(&H[(size_t)i * b + j], 2.f * acc[k], 2.f * acc[k + 1], 2.f * acc[k + 2],
                     2.f * acc[k + 3]);
          } else {
#pragma unroll
            for (int e = 0; e < 4; ++e)
              if (j + e < b && i <= j + e) red_add(&H[(size_t)i * b + j + e], 2.f * acc[k + e]);
          }
        }
#pragma unroll
        for (int k = 0; k < 128; ++k) {
          const int j = jbase + k;
          if (j < b && i < j) red_add(&H[(size_t)j * b + i], 2.f * acc[k]);
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512)
                 : "memory");
  }
  if (threadIdx.x == 0 && *abort_flag) atomicCAS(p.status, 0, (int)THANOS_ERR_TIMEOUT);
}

// x = h + m + l with three bf16 planes [3][n][b] (fp32 has 24 significant bits, 3 x 8); four
// consecutive features per thread (b and ldx are multiples of 8)
__global__ void split_planes_kernel(const float* __restrict__ X, int64_t ldx, int n, int b,
                                    __nv_bfloat16* __restrict__ planes) {
  const int b4 = b >> 2;
  const int64_t total4 = (int64_t)n * b4;
  const int64_t total = (int64_t)n * b;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total4; e += stride) {
    const int64_t t = e / b4;
    const int j = 4 * (int)(e - t * b4);
    const float4 xv = *reinterpret_cast<const float4*>(X + t * ldx + j);
    float x[4] = {xv.x, xv.y, xv.z, xv.w};
    const int64_t o = t * b + j;
#pragma unroll
    for (int pl = 0; pl < 3; ++pl) {
      __nv_bfloat16 hb[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        hb[k] = __float2bfloat16_rn(x[k]);
        x[k] -= __bfloat162float(hb[k]);
      }
      uint2 pk;
      pk.x = (uint32_t)__bfloat16_as_ushort(hb[0]) | ((uint32_t)__bfloat16_as_ushort(hb[1]) << 16);
      pk.y = (uint32_t)__bfloat16_as_ushort(hb[2]) | ((uint32_t)__bfloat16_as_ushort(hb[3]) << 16);
      *reinterpret_cast<uint2*>(planes + (int64_t)pl * total + o) = pk;
    }
  }
}

thanos_status_t launch_tc(float* H, int b, const __nv_bfloat16* base, int64_t ld_elems, int n_tok,
                          int planes, int64_t plane_stride_elems, int32_t* status,
                          cudaStream_t stream, bool one_slice) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return THANOS_ERR_CUDA;
  CUtensorMap tmap;
  cuuint64_t gdim[3] = {(cuuint64_t)b, (cuuint64_t)n_tok, (cuuint64_t)planes};
  cuuint64_t gstr[2] = {(cuuint64_t)ld_elems * 2, (cuuint64_t)plane_stride_elems * 2};
  const bool p3 = planes == 3;
  const int BK = p3 ? Geo<true>::BK : Geo<false>::BK;
  const int FLUSH_STAGES = p3 ? Geo<true>::FLUSH_STAGES : Geo<false>::FLUSH_STAGES;
  cuuint32_t box[3] = {64, (cuuint32_t)BK, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  if (enc(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<__nv_bfloat16*>(base), gdim, gstr,
          box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return THANOS_ERR_CUDA;

  Params p;
  p.H = H;
  p.status = status;
  p.b = b;
  p.n_tok = n_tok;
  p.nI = (b + TM - 1) / TM;
  p.nJ = (b + TN - 1) / TN;
  int tiles = 0;
  for (int J = 0; J < p.nJ; ++J) tiles += (2 * J + 2 < p.nI) ? 2 * J + 2 : p.nI;
  p.n_tiles = tiles;
  // token slices: pick the count (each slice >= 2048 tokens) that wastes the least of the last
  // wave of CTAs
  const int G = sm_count();
  // fewest slices whose last wave wastes at most 3 percent more than the best count does:
  // longer slices mean fewer write-outs of a tile
  int max_s = n_tok / 2048;
  if (max_s < 1) max_s = 1;
  if (max_s > 16) max_s = 16;
  double eff_of[17];
  double best_eff = 0.0;
  for (int s = 1; s <= max_s; ++s) {
    const long long units = (long long)tiles * s;
    const long long waves = (units + G - 1) / G;
    eff_of[s] = (double)units / (double)(waves * G);
    if (eff_of[s] > best_eff) best_eff = eff_of[s];
  }
  int best_s = 1;
  // one slice: every entry of H then receives exactly one addend per launch (fixed summation order)
  while (!one_slice && best_s < max_s && eff_of[best_s] < best_eff - 0.03) ++best_s;
  int st = (n_tok + best_s - 1) / best_s;
  st = (st + FLUSH_STAGES * BK - 1) / (FLUSH_STAGES * BK) * (FLUSH_STAGES * BK);
  p.slice_tokens = st;
  p.n_slices = (n_tok + st - 1) / st;
  if (planes == 1) {
    p.n_combo = 1;
    for (int i = 0; i < 6; ++i) p.plane_a[i] = p.plane_b[i] = 0;
  } else {
    p.n_combo = 6;
    const int pa[6] = {0, 0, 1, 0, 2, 1};
    const int pb[6] = {0, 1, 0, 2, 0, 1};
    for (int i = 0; i < 6; ++i) {
      p.plane_a[i] = pa[i];
      p.plane_b[i] = pb[i];
    }
  }
  long long units = (long long)p.n_tiles * p.n_slices;
  int grid = (int)(units < G ? units : G);
  if (p3) {
    static std::atomic<unsigned long long> done{0};
    THANOS_CUDA(ensure_max_dyn_smem(hessian_tc_kernel<true>, (int)Geo<true>::SMEM_BYTES, done));
    hessian_tc_kernel<true><<<grid, NTHREADS, Geo<true>::SMEM_BYTES, stream>>>(tmap, p);
  } else {
    static std::atomic<unsigned long long> done{0};
    THANOS_CUDA(ensure_max_dyn_smem(hessian_tc_kernel<false>, (int)Geo<false>::SMEM_BYTES, done));
    hessian_tc_kernel<false><<<grid, NTHREADS, Geo<false>::SMEM_BYTES, stream>>>(tmap, p);
  }
  THANOS_CHECK_LAUNCH();
  return THANOS_OK;
}

// Tokens of fp32 input split into planes per pass: as many as fit 2^28 plane bytes (a launch over a
// longer chunk has more token slices to fill the SMs with, which narrow layers need), between 8192
// and 65536 and a multiple of 512.
int64_t split_chunk_tokens(int64_t b) {
  int64_t t = ((int64_t)1 << 28) / (6 * b);
  t = t / 512 * 512;
  if (t < 8192) t = 8192;
  if (t > 65536) t = 65536;
  return t;
}

}  // namespace

bool hessian_tc2_supported(int64_t b, int64_t n_tok);
thanos_status_t launch_hessian_tc2(float* H, int b, const __nv_bfloat16* base, int64_t ld_elems,
                                   int n_tok, int32_t* status, cudaStream_t stream, bool one_slice);

size_t hessian_tc_workspace_bytes(int64_t b, thanos_dtype_t dtype) {
  size_t w = 256;  // status word
  if (dtype == THANOS_F32)
    w += round_up((size_t)3 * (size_t)split_chunk_tokens(b) * b * sizeof(__nv_bfloat16), 256);
  return w;
}

bool hessian_tc_supported(int64_t b, int64_t n_tok) { return b >= 256 && n_tok >= 64; }

thanos_status_t hessian_accumulate_tc(float* H, int64_t b, const void* X, thanos_dtype_t xdtype,
                                      int64_t n_tok, int64_t ldx, void* workspace,
                                      cudaStream_t stream, bool ordered) {
  int32_t* status = static_cast<int32_t*>(workspace);
  THANOS_CUDA(cudaMemsetAsync(status, 0, 16, stream));
  if (xdtype == THANOS_BF16) {
    // one launch covers at most 2^22 tokens (keeps every tensor-map stride below 2^40 bytes)
    const int64_t step = (int64_t)1 << 22;
    for (int64_t t0 = 0; t0 < n_tok; t0 += step) {
      int64_t n = n_tok - t0 < step ? n_tok - t0 : step;
      if (hessian_tc2_supported(b, n)) {  // CTA pairs; falls through if they cannot be scheduled
        thanos_status_t st2 = launch_hessian_tc2(
            H, (int)b, static_cast<const __nv_bfloat16*>(X) + t0 * ldx, ldx, (int)n, status, stream,
            ordered);
        if (st2 == THANOS_OK) continue;
        if (st2 != THANOS_ERR_SHAPE) return st2;
      }
      THANOS_TRY(launch_tc(H, (int)b, static_cast<const __nv_bfloat16*>(X) + t0 * ldx, ldx, (int)n,
                           1, n * ldx, status, stream, ordered));
    }
    return THANOS_OK;
  }
  __nv_bfloat16* planes = reinterpret_cast<__nv_bfloat16*>(static_cast<char*>(workspace) + 256);
  const int64_t chunk = split_chunk_tokens(b);
  for (int64_t t0 = 0; t0 < n_tok; t0 += chunk) {
    int n = (int)(n_tok - t0 < chunk ? n_tok - t0 : chunk);
    split_planes_kernel<<<NUM_SMS * 8, 256, 0, stream>>>(static_cast<const float*>(X) + t0 * ldx, ldx,
                                                     n, (int)b, planes);
    THANOS_CHECK_LAUNCH();
    THANOS_TRY(launch_tc(H, (int)b, planes, b, n, 3, (int64_t)n * b, status, stream, ordered));
  }
  return THANOS_OK;
}

}  // namespace thanos
