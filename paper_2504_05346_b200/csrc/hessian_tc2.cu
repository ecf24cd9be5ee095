// H += 2 X^T X on the 5th-generation tensor cores with CTA pairs (Section 3.2: H = 2 X X^T).
//
// A cluster of two CTAs (two SMs) owns a 256 x 256 tile of H.  CTA r of the pair holds rows
// 128 r .. 128 r + 127 of the tile in its tensor memory; per 64-token stage it loads only its own
// 128 features of the row block and 128 features of the column block (32 KB instead of the 48 KB
// a lone CTA needs for a 128 x 256 tile), and one tcgen05.mma.cta_group::2 of 256 x 256 x 16
// reads the operand halves from both CTAs' shared memory.  Shared-memory traffic per SM (TMA
// writes plus tensor-core reads) drops from 192 to 128 bytes per clock at full tensor rate.
// Roles per CTA:
//   warp 0      TMA producer (6-stage ring); transaction bytes of both CTAs land on the barrier of
//               the pair's first CTA
//   warp 1      first CTA: MMA issuer for the pair; second CTA: idle apart from TMEM alloc / free
//   warps 2..9  accumulation and write-out, as in the one-CTA kernel (registers promoted every
//               512 tokens, 2 * acc added to H[i, j] and to the mirror H[j, i])
// On diagonal tiles the row features are the column features, so only one half is loaded.
// Every mbarrier wait is bounded: on expiry the CTA raises an abort flag, the status word gets
// THANOS_ERR_TIMEOUT, the roles drain, the pair meets at the final cluster barrier and frees TMEM.
#include "tc_common.cuh"

namespace thanos {

namespace {

using namespace tc;

constexpr int TT = 256;           // tile edge of the pair
constexpr int BK = 64;            // tokens per pipeline stage
constexpr int STAGES = 6;
constexpr int FLUSH_STAGES = 8;   // TMEM accumulator drained every 8 stages = 512 tokens
constexpr int BOX_BYTES = 64 * BK * 2;        // one 64-feature x 64-token bf16 box
constexpr int STAGE_BYTES = 4 * BOX_BYTES;    // 2 boxes of the column half, 2 of the row half
constexpr int A_OFFSET = 2 * BOX_BYTES;
constexpr int NTHREADS = 320;
constexpr size_t SMEM_BYTES = (size_t)STAGES * STAGE_BYTES + 1024 /*align*/ + 256 /*barriers*/;

struct Params2 {
  float* H;
  int32_t* status;
  int b;
  int n_tok;
  int n_tiles;         // 256-blocks pairs (I <= J)
  int n_slices;
  int slice_tokens;    // multiple of BK
  int sb;              // super-block edge in tiles
};

// TMA tile load of a CTA pair: the bytes are counted on the barrier at `bar_cluster_addr`
// (the first CTA's), the data lands in this CTA's shared memory.
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* map,
                                                 uint32_t bar_cluster_addr, int x, int y, int z) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%3, %4, %5}], [%2];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(bar_cluster_addr), "r"(x), "r"(y), "r"(z)
      : "memory");
}
// MN-major bf16 operand stored as 64-feature x 64-token boxes with the 128-byte swizzle (see the
// one-CTA kernel): 8 tokens per 1024-byte atom, the next 64 features one box further.
__device__ __forceinline__ uint64_t make_desc2(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)((uint32_t)BOX_BYTES >> 4) << 16;
  d |= (uint64_t)(1024u >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
// kind::f16: D fp32, A and B bf16, both MN-major, M = 256 (over the pair), N = 256.
__device__ __forceinline__ uint32_t make_idesc2() {
  uint32_t d = 0;
  d |= 1u << 4;
  d |= 1u << 7;
  d |= 1u << 10;
  d |= 1u << 15;
  d |= 1u << 16;
  d |= (uint32_t)(TT >> 3) << 17;
  d |= (uint32_t)(TT >> 4) << 24;
  return d;
}

struct Unit2 {
  int I, J, t0, nst;
  bool diag;
};
// Tiles are numbered super-block by super-block (SB x SB tiles, upper triangle of super-blocks in
// column order): the pairs that run at the same time then share a handful of feature blocks of
// the same token slice, which the L2 serves -- in plain column order a wave of tiles spans most
// row blocks of a wide layer and every wave re-reads most of X from DRAM.
__device__ __forceinline__ Unit2 decode_unit2(const Params2& p, int u) {
  Unit2 r;
  int tile = u % p.n_tiles;
  const int slice = u / p.n_tiles;
  const int nT = (p.b + TT - 1) / TT;
  const int SB = p.sb;
  const int nS = (nT + SB - 1) / SB;
  int I = 0, J = 0;
  for (int SJ = 0; SJ < nS; ++SJ) {
    const int wj = min(SB, nT - SJ * SB);
    bool found = false;
    for (int SI = 0; SI <= SJ; ++SI) {
      const int wi = min(SB, nT - SI * SB);
      const int size = SI == SJ ? (wj * (wj + 1)) / 2 : wi * wj;
      if (tile < size) {
        int di, dj;
        if (SI == SJ) {
          dj = 0;
          while (tile > dj) {  // column dj of the triangle has dj + 1 tiles
            tile -= dj + 1;
            ++dj;
          }
          di = tile;
        } else {
          di = tile / wj;
          dj = tile - di * wj;
        }
        I = SI * SB + di;
        J = SJ * SB + dj;
        found = true;
        break;
      }
      tile -= size;
    }
    if (found) break;
  }
  r.I = I;
  r.J = J;
  r.diag = I == J;
  r.t0 = slice * p.slice_tokens;
  int t1 = r.t0 + p.slice_tokens;
  if (t1 > p.n_tok) t1 = p.n_tok;
  r.nst = (t1 - r.t0 + BK - 1) / BK;
  if (r.nst < 0) r.nst = 0;
  return r;
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NTHREADS, 1)
hessian_tc2_kernel(const __grid_constant__ CUtensorMap tmap, const Params2 p) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)STAGES * STAGE_BYTES);
  // bars[0..5] full (used in the first CTA), [6..11] empty, [12..13] tmem full,
  // [14..15] tmem empty (used in the first CTA)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 16);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 17);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1;
  const int npairs = gridDim.x >> 1;
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t bar_base = smem_u32(bars);
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  auto tfull_bar = [&](int q) { return bar_base + 8u * (2 * STAGES + q); };
  auto tempty_bar = [&](int q) { return bar_base + 8u * (2 * STAGES + 2 + q); };

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int q = 0; q < 2; ++q) {
      mbar_init(tfull_bar(q), 1);
      mbar_init(tempty_bar(q), 16);  // 8 accumulation warps in each CTA of the pair
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(tmem_slot)),
                 "r"(512)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // both CTAs' barriers are initialised before anything signals them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int n_units = p.n_tiles * p.n_slices;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    int s = 0;
    uint32_t phase = 0;
    bool ok = true;
    for (int u = pair; u < n_units && ok; u += npairs) {
      const Unit2 un = decode_unit2(p, u);
      for (int ks = 0; ks < un.nst && ok; ++ks) {
        ok = mbar_wait(empty_bar(s), phase ^ 1u, abort_flag);
        if (ok && lane == 0) {
          const uint32_t dst = smem_base + (uint32_t)s * STAGE_BYTES;
          const uint32_t lead_bar = map_to_cta(full_bar(s), 0);
          const int y = un.t0 + ks * BK;
          // the first CTA announces the bytes of both CTAs
          if (rank == 0) mbar_expect_tx(full_bar(s), 2 * (un.diag ? 2 : 4) * BOX_BYTES);
          const int jb = un.J * TT + 128 * (int)rank;
#pragma unroll
          for (int i = 0; i < 2; ++i)
            tma_load_3d_pair(dst + i * BOX_BYTES, &tmap, lead_bar, jb + 64 * i, y, 0);
          if (!un.diag) {
            const int ib = un.I * TT + 128 * (int)rank;
#pragma unroll
            for (int i = 0; i < 2; ++i)
              tma_load_3d_pair(dst + A_OFFSET + i * BOX_BYTES, &tmap, lead_bar, ib + 64 * i, y, 0);
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
    // ------------------------------------------------------------ MMA issuer (first CTA only)
    if (rank == 0) {
      const uint32_t idesc = make_idesc2();
      int s = 0, q = 0;
      uint32_t phase = 0, tphase = 0;
      bool ok = true;
      for (int u = pair; u < n_units && ok; u += npairs) {
        const Unit2 un = decode_unit2(p, u);
        for (int g0 = 0; g0 < un.nst && ok; g0 += FLUSH_STAGES) {
          const int g1 = g0 + FLUSH_STAGES < un.nst ? g0 + FLUSH_STAGES : un.nst;
          ok = mbar_wait(tempty_bar(q), tphase ^ 1u, abort_flag);
          tc_fence_after();
          for (int kk = g0; kk < g1 && ok; ++kk) {
            ok = mbar_wait(full_bar(s), phase, abort_flag);
            tc_fence_after();
            if (ok && lane == 0) {
              const uint32_t sb = smem_base + (uint32_t)s * STAGE_BYTES;
              const uint32_t sa = un.diag ? sb : sb + A_OFFSET;
#pragma unroll
              for (int k4 = 0; k4 < BK / 16; ++k4) {
                const uint64_t adesc = make_desc2(sa + k4 * 2048);
                const uint64_t bdesc = make_desc2(sb + k4 * 2048);
                tc_mma_bf16_pair(tmem_base + (uint32_t)q * TT, adesc, bdesc, idesc,
                                 (kk > g0 || k4 > 0) ? 1u : 0u);
              }
              tc_commit_pair(empty_bar(s));
            }
            __syncwarp();
            if (++s == STAGES) {
              s = 0;
              phase ^= 1u;
            }
          }
          if (ok && lane == 0) tc_commit_pair(tfull_bar(q));
          __syncwarp();
          if (++q == 2) {
            q = 0;
            tphase ^= 1u;
          }
        }
      }
    }
  } else {
    // ------------------------------------------------------------ accumulate + write out
    const int ew = warp - 2;
    const int g = warp & 3;     // TMEM lane quarter this warp may read
    const int h = ew >> 2;      // column half
    const uint32_t lead_tempty[2] = {map_to_cta(tempty_bar(0), 0), map_to_cta(tempty_bar(1), 0)};
    int q = 0;
    uint32_t tphase = 0;
    bool ok = true;
    for (int u = pair; u < n_units && ok; u += npairs) {
      const Unit2 un = decode_unit2(p, u);
      float acc[128];
#pragma unroll
      for (int k = 0; k < 128; ++k) acc[k] = 0.f;
      for (int g0 = 0; g0 < un.nst && ok; g0 += FLUSH_STAGES) {
        ok = mbar_wait(tfull_bar(q), tphase, abort_flag);
        tc_fence_after();
        if (ok) {
          const uint32_t taddr = tmem_base + ((uint32_t)(32 * g) << 16) + (uint32_t)q * TT + h * 128;
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
        if (lane == 0) mbar_arrive_cluster(lead_tempty[q]);
        if (++q == 2) {
          q = 0;
          tphase ^= 1u;
        }
      }
      if (!ok || un.nst == 0) continue;
      const int i = un.I * TT + 128 * (int)rank + 32 * g + lane;
      const int jbase = un.J * TT + h * 128;
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

  // Neither CTA may leave (or free tensor memory) while its partner can still read its shared
  // memory, signal its barriers or write its tensor memory.
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512)
                 : "memory");
  }
  if (threadIdx.x == 0 && *abort_flag) atomicCAS(p.status, 0, (int)THANOS_ERR_TIMEOUT);
}

// Clusters of two that can be resident at once (the grid is sized to it, persistent pairs).
int max_active_pairs() {
  static std::atomic<int> cached_by_dev[64];  // 0 = not asked yet, else pairs + 1
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
  const int have = cached_by_dev[dev].load(std::memory_order_relaxed);
  if (have > 0) return have - 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * sm_count(), 1, 1);
  cfg.blockDim = dim3(NTHREADS, 1, 1);
  cfg.dynamicSmemBytes = SMEM_BYTES;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, hessian_tc2_kernel, &cfg) != cudaSuccess || n <= 0) {
    cudaGetLastError();
    n = 0;
  }
  cached_by_dev[dev].store(n + 1, std::memory_order_relaxed);
  return n;
}

}  // namespace

bool hessian_tc2_supported(int64_t b, int64_t n_tok) { return b >= 1024 && n_tok >= 512; }

// bf16 X [n_tok, b] (leading dimension ld_elems); returns THANOS_ERR_SHAPE when CTA pairs cannot
// be scheduled on this device (the caller then uses the one-CTA kernel).
thanos_status_t launch_hessian_tc2(float* H, int b, const __nv_bfloat16* base, int64_t ld_elems,
                                   int n_tok, int32_t* status, cudaStream_t stream, bool one_slice) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return THANOS_ERR_CUDA;
  {
    static std::atomic<unsigned long long> done{0};
    THANOS_CUDA(ensure_max_dyn_smem(hessian_tc2_kernel, (int)SMEM_BYTES, done));
  }
  const int G = max_active_pairs();
  if (G < 8) return THANOS_ERR_SHAPE;
  CUtensorMap tmap;
  cuuint64_t gdim[3] = {(cuuint64_t)b, (cuuint64_t)n_tok, 1};
  cuuint64_t gstr[2] = {(cuuint64_t)ld_elems * 2, (cuuint64_t)ld_elems * 2 * (cuuint64_t)n_tok};
  cuuint32_t box[3] = {64, (cuuint32_t)BK, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  if (enc(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<__nv_bfloat16*>(base), gdim, gstr,
          box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return THANOS_ERR_CUDA;
  Params2 p;
  p.H = H;
  p.status = status;
  p.b = b;
  p.n_tok = n_tok;
  const int nT = (b + TT - 1) / TT;
  p.n_tiles = nT * (nT + 1) / 2;
  p.sb = 8;  // 64 tiles per super-block: about one wave of the 74 pairs
  // token slices: the count (each slice >= 2048 tokens) that wastes the least of the last wave
  // fewest slices whose last wave wastes at most 3 percent more than the best count does:
  // longer slices mean fewer write-outs of a tile
  int max_s = n_tok / 2048;
  if (max_s < 1) max_s = 1;
  if (max_s > 16) max_s = 16;
  double eff_of[17];
  double best_eff = 0.0;
  for (int s = 1; s <= max_s; ++s) {
    const long long units = (long long)p.n_tiles * s;
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
  const long long units = (long long)p.n_tiles * p.n_slices;
  const int pairs = (int)(units < G ? units : G);
  hessian_tc2_kernel<<<2 * pairs, NTHREADS, SMEM_BYTES, stream>>>(tmap, p);
  THANOS_CHECK_LAUNCH();
  return THANOS_OK;
}

}  // namespace thanos
