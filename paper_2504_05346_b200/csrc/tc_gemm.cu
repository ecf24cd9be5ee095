// fp32-accurate GEMM on tcgen05: D = [D +] alpha * A * Bop with every operand given as three
// bf16 planes (see tc_gemm.cuh).
//
// One persistent CTA per SM over 128 x 128 output tiles.  Roles:
//   warp 0      TMA producer: per 64-wide k step the three planes of the A tile (128 rows x 64 k,
//               K-major, 128-byte swizzle) and of the B tile (K-major: 128 n x 64 k; MN-major:
//               two boxes of 64 n x 64 k) -- 96 KB per stage, two stages
//   warp 1      tcgen05.mma issuer: per stage 6 plane pairs x 4 MMAs of 128 x 128 x 16
//   warps 2..9  epilogue: TMEM -> registers -> 128 x 32 fp32 staging buffers in shared memory ->
//               TMA reduce-add (or store) into D; if asked, the result also split into bf16
//               planes for the next product
// TMEM: two 128 x 128 fp32 accumulators, so the epilogue of a tile overlaps the next tile's MMAs.
// Every wait is bounded (see tc_common.cuh); on expiry the status word gets THANOS_ERR_TIMEOUT.
//
// Large products run the same roles on CTA pairs (tc_gemm_pair_kernel below): 256 x 256 tiles,
// tcgen05.mma.cta_group::2, half the operand bytes per output element.
#include "tc_gemm.cuh"

#include "tc_common.cuh"

namespace thanos {

namespace {

using namespace tc;

constexpr int TM = 128;
constexpr int TN = 128;
constexpr int BK = 64;
constexpr int STAGES = 2;
constexpr int PLANE_TILE_BYTES = 128 * BK * 2;       // 16 KB: one plane of an operand tile
constexpr int STAGE_BYTES = 6 * PLANE_TILE_BYTES;    // A planes 0..2, then B planes 0..2
constexpr int B_OFFSET = 3 * PLANE_TILE_BYTES;
constexpr int NTHREADS = 320;
constexpr int STAGING_BYTES = 128 * 32 * 4;          // 16 KB: 128 rows x 32 fp32 columns of D
constexpr size_t SMEM_BYTES =
    (size_t)STAGES * STAGE_BYTES + 2 * STAGING_BYTES + 1024 /*align*/ + 256 /*barriers*/;
constexpr uint32_t TMEM_COLS = 256;

struct Params {
  float* D;
  __nv_bfloat16* Dp;
  int64_t ldd, d_batch, ldp, dp_plane, dp_batch;
  int32_t* status;
  int M, N, K, batch;
  int tiles_m, tiles_n;
  int b_kmajor, accumulate, upper_only, a_upper, b_upper;
  float alpha;
};

// K-major operand tile: rows of 64 bf16 (128 bytes), 8 rows per 1024-byte swizzle atom.
__device__ __forceinline__ uint64_t desc_kmajor(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;                 // leading offset: not used by swizzled K-major layouts
  d |= (uint64_t)(1024u >> 4) << 32;      // stride between 8-row groups
  d |= (uint64_t)1 << 46;                 // descriptor version for sm_100
  d |= (uint64_t)2 << 61;                 // 128-byte swizzle
  return d;
}
// MN-major operand tile made of 64 n x 64 k boxes: a k row is 128 bytes, 8 k rows per atom, the
// next 64 n are one box (8 KB) further.
__device__ __forceinline__ uint64_t desc_mnmajor(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)(8192u >> 4) << 16;
  d |= (uint64_t)(1024u >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
__device__ __forceinline__ uint32_t make_idesc(int b_kmajor) {
  uint32_t d = 0;
  d |= 1u << 4;    // D fp32
  d |= 1u << 7;    // A bf16
  d |= 1u << 10;   // B bf16
  if (!b_kmajor) d |= 1u << 16;  // B is MN-major (A is K-major: bit 15 clear)
  d |= (uint32_t)(TN >> 3) << 17;
  d |= (uint32_t)(TM >> 4) << 24;
  return d;
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar,
                                            int x, int y, int z, int w) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%3, %4, %5, %6}], [%2];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y), "r"(z), "r"(w)
      : "memory");
}

__device__ __forceinline__ void tma_reduce_add_3d(const CUtensorMap* map, uint32_t src, int x,
                                                  int y, int z) {
  asm volatile(
      "cp.reduce.async.bulk.tensor.3d.global.shared::cta.add.tile.bulk_group [%0, {%2, %3, %4}], [%1];" ::
          "l"(reinterpret_cast<uint64_t>(map)),
      "r"(src), "r"(x), "r"(y), "r"(z)
      : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, uint32_t src, int x, int y,
                                             int z) {
  asm volatile(
      "cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4}], [%1];" ::"l"(
          reinterpret_cast<uint64_t>(map)),
      "r"(src), "r"(x), "r"(y), "r"(z)
      : "memory");
}
__device__ __forceinline__ void named_bar_sync(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

struct Tile {
  int z, m0, n0;
  int ks0, ks1;  // k steps [ks0, ks1) that can hold non-zero products
  bool skip;
};
__device__ __forceinline__ Tile decode_tile(const Params& p, int t) {
  Tile r;
  const int per = p.tiles_m * p.tiles_n;
  r.z = t / per;
  const int rem = t - r.z * per;
  const int mi = rem / p.tiles_n;
  r.m0 = mi * TM;
  r.n0 = (rem - mi * p.tiles_n) * TN;
  r.skip = p.upper_only && (r.n0 + TN - 1 < r.m0);
  r.ks0 = p.a_upper ? r.m0 / BK : 0;
  r.ks1 = (p.K + BK - 1) / BK;
  if (p.b_upper) {
    const int lim = (r.n0 + TN + BK - 1) / BK;
    if (lim < r.ks1) r.ks1 = lim;
  }
  if (r.ks1 <= r.ks0) r.ks1 = r.ks0 + 1;  // at least one step so that the accumulator is defined
  return r;
}

__constant__ int c_plane_a[6] = {0, 0, 1, 0, 2, 1};
__constant__ int c_plane_b[6] = {0, 1, 0, 2, 0, 1};

__global__ void __launch_bounds__(NTHREADS, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB,
               const __grid_constant__ CUtensorMap mapD, const Params p) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* bars =
      reinterpret_cast<uint64_t*>(smem + (size_t)STAGES * STAGE_BYTES + 2 * STAGING_BYTES);
  // bars[0..1] full, [2..3] empty, [4..5] tmem full, [6..7] tmem empty
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 8);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 9);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t bar_base = smem_u32(bars);
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (2 + s); };
  auto tfull_bar = [&](int q) { return bar_base + 8u * (4 + q); };
  auto tempty_bar = [&](int q) { return bar_base + 8u * (6 + q); };

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
                 "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int n_tiles = p.tiles_m * p.tiles_n * p.batch;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    int s = 0;
    uint32_t phase = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x) {
      const Tile tl = decode_tile(p, t);
      if (tl.skip) continue;
      for (int ks = tl.ks0; ks < tl.ks1 && ok; ++ks) {
        ok = mbar_wait(empty_bar(s), phase ^ 1u, abort_flag);
        if (ok && lane == 0) {
          const uint32_t dst = smem_base + (uint32_t)s * STAGE_BYTES;
          const int k0 = ks * BK;
          mbar_expect_tx(full_bar(s), STAGE_BYTES);
#pragma unroll
          for (int pl = 0; pl < 3; ++pl)
            tma_load_4d(dst + pl * PLANE_TILE_BYTES, &mapA, full_bar(s), k0, tl.m0, pl, tl.z);
          if (p.b_kmajor) {
#pragma unroll
            for (int pl = 0; pl < 3; ++pl)
              tma_load_4d(dst + B_OFFSET + pl * PLANE_TILE_BYTES, &mapB, full_bar(s), k0, tl.n0, pl,
                          tl.z);
          } else {
#pragma unroll
            for (int pl = 0; pl < 3; ++pl) {
              tma_load_4d(dst + B_OFFSET + pl * PLANE_TILE_BYTES, &mapB, full_bar(s), tl.n0, k0, pl,
                          tl.z);
              tma_load_4d(dst + B_OFFSET + pl * PLANE_TILE_BYTES + 8192, &mapB, full_bar(s),
                          tl.n0 + 64, k0, pl, tl.z);
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
    const uint32_t idesc = make_idesc(p.b_kmajor);
    int s = 0, q = 0;
    uint32_t phase = 0, tphase = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x) {
      const Tile tl = decode_tile(p, t);
      if (tl.skip) continue;
      ok = mbar_wait(tempty_bar(q), tphase ^ 1u, abort_flag);
      tc_fence_after();
      for (int ks = tl.ks0; ks < tl.ks1 && ok; ++ks) {
        ok = mbar_wait(full_bar(s), phase, abort_flag);
        tc_fence_after();
        if (ok && lane == 0) {
          const uint32_t sa = smem_base + (uint32_t)s * STAGE_BYTES;
          const uint32_t sb = sa + B_OFFSET;
#pragma unroll
          for (int cb = 0; cb < 6; ++cb) {
            const uint32_t pa = sa + (uint32_t)c_plane_a[cb] * PLANE_TILE_BYTES;
            const uint32_t pb = sb + (uint32_t)c_plane_b[cb] * PLANE_TILE_BYTES;
#pragma unroll
            for (int k4 = 0; k4 < BK / 16; ++k4) {
              const uint64_t adesc = desc_kmajor(pa + k4 * 32);
              const uint64_t bdesc =
                  p.b_kmajor ? desc_kmajor(pb + k4 * 32) : desc_mnmajor(pb + k4 * 2048);
              tc_mma_bf16(tmem_base + (uint32_t)q * TN, adesc, bdesc, idesc,
                          (ks > tl.ks0 || cb > 0 || k4 > 0) ? 1u : 0u);
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
  } else {
    // ------------------------------------------------------------ epilogue
    // Warp w reads TMEM lanes 32 (w & 3) .. +31 (one output row per thread) and the column half
    // h = (w - 2) / 4, 32 columns at a time.  The four warps of a half share one 128 x 32 fp32
    // staging buffer (128-byte swizzle); one thread of the half hands it to TMA, which adds it to
    // D (or stores it) with full-line accesses and no read in the SM.
    const int g = warp & 3;
    const int h = (warp - 2) >> 2;
    const bool issuer = g == 0 && lane == 0;
    unsigned char* stg = smem + (size_t)STAGES * STAGE_BYTES + (size_t)h * STAGING_BYTES;
    const uint32_t stg_addr = smem_u32(stg);
    const int r_in_tile = 32 * g + lane;
    int q = 0;
    uint32_t tphase = 0;
    bool ok = true;
    // After a failed wait the warp keeps walking the tiles (the waits then return at once) so
    // that the four warps of a half always meet at the same named barriers.
    for (int t = blockIdx.x; t < n_tiles; t += gridDim.x) {
      const Tile tl = decode_tile(p, t);
      if (tl.skip) continue;
      const int row = tl.m0 + r_in_tile;
      ok = ok && mbar_wait(tfull_bar(q), tphase, abort_flag);
      tc_fence_after();
      {
        const uint32_t taddr =
            tmem_base + ((uint32_t)(32 * g) << 16) + (uint32_t)q * TN + (uint32_t)h * 64;
#pragma unroll 1
        for (int cc = 0; cc < 2; ++cc) {
          uint32_t v[32];
          if (ok) {
            tc_ld32(taddr + cc * 32, v);
            tc_wait_ld();
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = 0u;
          }
          const int cbase = tl.n0 + 64 * h + 32 * cc;
          if (p.D || p.Dp) {
            // the buffer is free once TMA has read the previous chunk out of it
            if (issuer) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
            named_bar_sync(1 + 2 * h, 128);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              float4 o;
              o.x = p.alpha * __uint_as_float(v[4 * j + 0]);
              o.y = p.alpha * __uint_as_float(v[4 * j + 1]);
              o.z = p.alpha * __uint_as_float(v[4 * j + 2]);
              o.w = p.alpha * __uint_as_float(v[4 * j + 3]);
              *reinterpret_cast<float4*>(stg + r_in_tile * 128 + ((j ^ (r_in_tile & 7)) << 4)) = o;
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            named_bar_sync(2 + 2 * h, 128);
            if (issuer && ok && cbase < p.N && p.D) {
              if (p.accumulate) tma_reduce_add_3d(&mapD, stg_addr, cbase, tl.m0, tl.z);
              else tma_store_3d(&mapD, stg_addr, cbase, tl.m0, tl.z);
              asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            }
          }
          if (p.Dp && ok) {
            // Planes of the result from the staging buffer: every warp instruction covers four
            // rows of 32 columns (64 contiguous bytes per row and plane) instead of one 8-byte
            // piece in each of 32 rows.  The buffer is not reused before the next chunk's barrier.
            const int tih = 32 * g + lane;
            const int c4 = tih & 7;
            const int col = cbase + 4 * c4;
#pragma unroll
            for (int it = 0; it < 8; ++it) {
              const int rr = (tih >> 3) + 16 * it;
              const int grow = tl.m0 + rr;
              if (grow >= p.M || col >= p.N) continue;
              const float4 sv =
                  *reinterpret_cast<const float4*>(stg + rr * 128 + ((c4 ^ (rr & 7)) << 4));
              float o[4] = {sv.x, sv.y, sv.z, sv.w};
              __nv_bfloat16* pr = p.Dp + (int64_t)tl.z * p.dp_batch + (int64_t)grow * p.ldp;
              if (col + 3 < p.N) {
#pragma unroll
                for (int pl = 0; pl < 3; ++pl) {
                  __nv_bfloat16 hb[4];
#pragma unroll
                  for (int e = 0; e < 4; ++e) {
                    hb[e] = __float2bfloat16_rn(o[e]);
                    o[e] -= __bfloat162float(hb[e]);
                  }
                  uint2 pk;
                  pk.x = (uint32_t)__bfloat16_as_ushort(hb[0]) |
                         ((uint32_t)__bfloat16_as_ushort(hb[1]) << 16);
                  pk.y = (uint32_t)__bfloat16_as_ushort(hb[2]) |
                         ((uint32_t)__bfloat16_as_ushort(hb[3]) << 16);
                  *reinterpret_cast<uint2*>(pr + (int64_t)pl * p.dp_plane + col) = pk;
                }
              } else {
                for (int e = 0; e < 4 && col + e < p.N; ++e) {
                  float val = o[e];
                  for (int pl = 0; pl < 3; ++pl) {
                    const __nv_bfloat16 hb = __float2bfloat16_rn(val);
                    pr[(int64_t)pl * p.dp_plane + col + e] = hb;
                    val -= __bfloat162float(hb);
                  }
                }
              }
            }
          }
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
    // every bulk store of this thread has to be complete before the kernel ends
    if (issuer) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                 "r"(TMEM_COLS)
                 : "memory");
  }
  if (threadIdx.x == 0 && *abort_flag && p.status) atomicCAS(p.status, 0, (int)THANOS_ERR_TIMEOUT);
}

// ---------------------------------------------------------------------------------------------
// The same product on CTA pairs: a cluster of two CTAs owns a 256 x 256 output tile.  CTA r of the
// pair loads rows 128 r .. 128 r + 127 of the A tile and columns 128 r .. 128 r + 127 of the B
// tile (96 KB per 64-wide k step, as above), one tcgen05.mma.cta_group::2 of 256 x 256 x 16 reads
// both halves from the two CTAs' shared memory, and CTA r's tensor memory holds rows 128 r .. of
// the accumulator (two accumulators of 256 columns).  Per output element the pair moves half the
// operand bytes of two lone CTAs, which is what holds the lone-CTA kernel back on large products.
// Barriers: the transaction bytes of both CTAs land on the first CTA's "full" barriers; commits
// are multicast to both CTAs' "empty" and "accumulator full" barriers; the eight epilogue warps of
// each CTA arrive on the first CTA's "accumulator empty" barriers.
constexpr int PTM = 256;
constexpr int PTN = 256;
constexpr uint32_t PAIR_TMEM_COLS = 512;

__device__ __forceinline__ void tma_load_4d_pair(uint32_t dst, const CUtensorMap* map,
                                                 uint32_t bar_cluster_addr, int x, int y, int z,
                                                 int w) {
  asm volatile(
      "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%3, %4, %5, %6}], [%2];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(bar_cluster_addr), "r"(x), "r"(y), "r"(z), "r"(w)
      : "memory");
}
__device__ __forceinline__ uint32_t make_idesc_pair(int b_kmajor) {
  uint32_t d = 0;
  d |= 1u << 4;    // D fp32
  d |= 1u << 7;    // A bf16
  d |= 1u << 10;   // B bf16
  if (!b_kmajor) d |= 1u << 16;  // B is MN-major (A is K-major: bit 15 clear)
  d |= (uint32_t)(PTN >> 3) << 17;
  d |= (uint32_t)(PTM >> 4) << 24;
  return d;
}
// p.tiles_m / p.tiles_n count 256 x 256 tiles here
__device__ __forceinline__ Tile decode_pair_tile(const Params& p, int t) {
  Tile r;
  const int per = p.tiles_m * p.tiles_n;
  r.z = t / per;
  const int rem = t - r.z * per;
  const int mi = rem / p.tiles_n;
  r.m0 = mi * PTM;
  r.n0 = (rem - mi * p.tiles_n) * PTN;
  r.skip = p.upper_only && (r.n0 + PTN - 1 < r.m0);
  r.ks0 = p.a_upper ? r.m0 / BK : 0;
  r.ks1 = (p.K + BK - 1) / BK;
  if (p.b_upper) {
    const int lim = (r.n0 + PTN + BK - 1) / BK;
    if (lim < r.ks1) r.ks1 = lim;
  }
  if (r.ks1 <= r.ks0) r.ks1 = r.ks0 + 1;
  return r;
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NTHREADS, 1)
tc_gemm_pair_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB,
                    const __grid_constant__ CUtensorMap mapD, const Params p) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* bars =
      reinterpret_cast<uint64_t*>(smem + (size_t)STAGES * STAGE_BYTES + 2 * STAGING_BYTES);
  // bars[0..1] full (used in the first CTA), [2..3] empty, [4..5] tmem full,
  // [6..7] tmem empty (used in the first CTA)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 8);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 9);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1;
  const int npairs = gridDim.x >> 1;
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t bar_base = smem_u32(bars);
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (2 + s); };
  auto tfull_bar = [&](int q) { return bar_base + 8u * (4 + q); };
  auto tempty_bar = [&](int q) { return bar_base + 8u * (6 + q); };

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int q = 0; q < 2; ++q) {
      mbar_init(tfull_bar(q), 1);
      mbar_init(tempty_bar(q), 16);  // 8 epilogue warps in each CTA of the pair
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(tmem_slot)),
                 "r"(PAIR_TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // both CTAs' barriers are initialised before anything signals them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int n_tiles = p.tiles_m * p.tiles_n * p.batch;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    int s = 0;
    uint32_t phase = 0;
    bool ok = true;
    for (int t = pair; t < n_tiles && ok; t += npairs) {
      const Tile tl = decode_pair_tile(p, t);
      if (tl.skip) continue;
      const int mrow = tl.m0 + 128 * (int)rank;
      const int ncol = tl.n0 + 128 * (int)rank;
      for (int ks = tl.ks0; ks < tl.ks1 && ok; ++ks) {
        ok = mbar_wait(empty_bar(s), phase ^ 1u, abort_flag);
        if (ok && lane == 0) {
          const uint32_t dst = smem_base + (uint32_t)s * STAGE_BYTES;
          const uint32_t lead_bar = map_to_cta(full_bar(s), 0);
          const int k0 = ks * BK;
          // the first CTA announces the bytes of both CTAs
          if (rank == 0) mbar_expect_tx(full_bar(s), 2 * STAGE_BYTES);
#pragma unroll
          for (int pl = 0; pl < 3; ++pl)
            tma_load_4d_pair(dst + pl * PLANE_TILE_BYTES, &mapA, lead_bar, k0, mrow, pl, tl.z);
          if (p.b_kmajor) {
#pragma unroll
            for (int pl = 0; pl < 3; ++pl)
              tma_load_4d_pair(dst + B_OFFSET + pl * PLANE_TILE_BYTES, &mapB, lead_bar, k0, ncol, pl,
                               tl.z);
          } else {
#pragma unroll
            for (int pl = 0; pl < 3; ++pl) {
              tma_load_4d_pair(dst + B_OFFSET + pl * PLANE_TILE_BYTES, &mapB, lead_bar, ncol, k0, pl,
                               tl.z);
              tma_load_4d_pair(dst + B_OFFSET + pl * PLANE_TILE_BYTES + 8192, &mapB, lead_bar,
                               ncol + 64, k0, pl, tl.z);
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
    // ------------------------------------------------------------ MMA issuer (first CTA only)
    if (rank == 0) {
      const uint32_t idesc = make_idesc_pair(p.b_kmajor);
      int s = 0, q = 0;
      uint32_t phase = 0, tphase = 0;
      bool ok = true;
      for (int t = pair; t < n_tiles && ok; t += npairs) {
        const Tile tl = decode_pair_tile(p, t);
        if (tl.skip) continue;
        ok = mbar_wait(tempty_bar(q), tphase ^ 1u, abort_flag);
        tc_fence_after();
        for (int ks = tl.ks0; ks < tl.ks1 && ok; ++ks) {
          ok = mbar_wait(full_bar(s), phase, abort_flag);
          tc_fence_after();
          if (ok && lane == 0) {
            const uint32_t sa = smem_base + (uint32_t)s * STAGE_BYTES;
            const uint32_t sb = sa + B_OFFSET;
#pragma unroll
            for (int cb = 0; cb < 6; ++cb) {
              const uint32_t pa = sa + (uint32_t)c_plane_a[cb] * PLANE_TILE_BYTES;
              const uint32_t pb = sb + (uint32_t)c_plane_b[cb] * PLANE_TILE_BYTES;
#pragma unroll
              for (int k4 = 0; k4 < BK / 16; ++k4) {
                const uint64_t adesc = desc_kmajor(pa + k4 * 32);
                const uint64_t bdesc =
                    p.b_kmajor ? desc_kmajor(pb + k4 * 32) : desc_mnmajor(pb + k4 * 2048);
                tc_mma_bf16_pair(tmem_base + (uint32_t)q * PTN, adesc, bdesc, idesc,
                                 (ks > tl.ks0 || cb > 0 || k4 > 0) ? 1u : 0u);
              }
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
  } else {
    // ------------------------------------------------------------ epilogue
    // As in the lone-CTA kernel: warp w reads TMEM lanes 32 (w & 3) .. +31 (one output row per
    // thread) and the column half h = (w - 2) / 4 of the CTA's 128 x 256 part, 32 columns at a time.
    const int g = warp & 3;
    const int h = (warp - 2) >> 2;
    const bool issuer = g == 0 && lane == 0;
    unsigned char* stg = smem + (size_t)STAGES * STAGE_BYTES + (size_t)h * STAGING_BYTES;
    const uint32_t stg_addr = smem_u32(stg);
    const int r_in_tile = 32 * g + lane;
    const uint32_t lead_tempty[2] = {map_to_cta(tempty_bar(0), 0), map_to_cta(tempty_bar(1), 0)};
    int q = 0;
    uint32_t tphase = 0;
    bool ok = true;
    for (int t = pair; t < n_tiles; t += npairs) {
      const Tile tl = decode_pair_tile(p, t);
      if (tl.skip) continue;
      const int m0 = tl.m0 + 128 * (int)rank;  // first row of this CTA's part
      ok = ok && mbar_wait(tfull_bar(q), tphase, abort_flag);
      tc_fence_after();
      {
        const uint32_t taddr =
            tmem_base + ((uint32_t)(32 * g) << 16) + (uint32_t)q * PTN + (uint32_t)h * 128;
#pragma unroll 1
        for (int cc = 0; cc < 4; ++cc) {
          uint32_t v[32];
          if (ok) {
            tc_ld32(taddr + cc * 32, v);
            tc_wait_ld();
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = 0u;
          }
          const int cbase = tl.n0 + 128 * h + 32 * cc;
          if (p.D || p.Dp) {
            // the buffer is free once TMA has read the previous chunk out of it
            if (issuer) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
            named_bar_sync(1 + 2 * h, 128);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              float4 o;
              o.x = p.alpha * __uint_as_float(v[4 * j + 0]);
              o.y = p.alpha * __uint_as_float(v[4 * j + 1]);
              o.z = p.alpha * __uint_as_float(v[4 * j + 2]);
              o.w = p.alpha * __uint_as_float(v[4 * j + 3]);
              *reinterpret_cast<float4*>(stg + r_in_tile * 128 + ((j ^ (r_in_tile & 7)) << 4)) = o;
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            named_bar_sync(2 + 2 * h, 128);
            if (issuer && ok && cbase < p.N && m0 < p.M && p.D) {
              if (p.accumulate) tma_reduce_add_3d(&mapD, stg_addr, cbase, m0, tl.z);
              else tma_store_3d(&mapD, stg_addr, cbase, m0, tl.z);
              asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            }
          }
          if (p.Dp && ok) {
            const int tih = 32 * g + lane;
            const int c4 = tih & 7;
            const int col = cbase + 4 * c4;
#pragma unroll
            for (int it = 0; it < 8; ++it) {
              const int rr = (tih >> 3) + 16 * it;
              const int grow = m0 + rr;
              if (grow >= p.M || col >= p.N) continue;
              const float4 sv =
                  *reinterpret_cast<const float4*>(stg + rr * 128 + ((c4 ^ (rr & 7)) << 4));
              float o[4] = {sv.x, sv.y, sv.z, sv.w};
              __nv_bfloat16* pr = p.Dp + (int64_t)tl.z * p.dp_batch + (int64_t)grow * p.ldp;
              if (col + 3 < p.N) {
#pragma unroll
                for (int pl = 0; pl < 3; ++pl) {
                  __nv_bfloat16 hb[4];
#pragma unroll
                  for (int e = 0; e < 4; ++e) {
                    hb[e] = __float2bfloat16_rn(o[e]);
                    o[e] -= __bfloat162float(hb[e]);
                  }
                  uint2 pk;
                  pk.x = (uint32_t)__bfloat16_as_ushort(hb[0]) |
                         ((uint32_t)__bfloat16_as_ushort(hb[1]) << 16);
                  pk.y = (uint32_t)__bfloat16_as_ushort(hb[2]) |
                         ((uint32_t)__bfloat16_as_ushort(hb[3]) << 16);
                  *reinterpret_cast<uint2*>(pr + (int64_t)pl * p.dp_plane + col) = pk;
                }
              } else {
                for (int e = 0; e < 4 && col + e < p.N; ++e) {
                  float val = o[e];
                  for (int pl = 0; pl < 3; ++pl) {
                    const __nv_bfloat16 hb = __float2bfloat16_rn(val);
                    pr[(int64_t)pl * p.dp_plane + col + e] = hb;
                    val -= __bfloat162float(hb);
                  }
                }
              }
            }
          }
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
    // every bulk store of this thread has to be complete before the kernel ends
    if (issuer) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  }

  // Neither CTA may leave (or free tensor memory) while its partner can still read its shared
  // memory, signal its barriers or write its tensor memory.
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                 "r"(PAIR_TMEM_COLS)
                 : "memory");
  }
  if (threadIdx.x == 0 && *abort_flag && p.status) atomicCAS(p.status, 0, (int)THANOS_ERR_TIMEOUT);
}

// Clusters of two of the pair kernel that can be resident at once (cached per device; 0 if the
// device cannot schedule them).
int max_active_gemm_pairs() {
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
  if (cudaOccupancyMaxActiveClusters(&n, tc_gemm_pair_kernel, &cfg) != cudaSuccess || n <= 0) {
    cudaGetLastError();
    n = 0;
  }
  cached_by_dev[dev].store(n + 1, std::memory_order_relaxed);
  return n;
}

bool make_map(CUtensorMap* map, const __nv_bfloat16* base, int64_t inner, int64_t rows, int64_t ld,
              int64_t plane_stride, int64_t batch, int64_t batch_stride, int box_inner,
              int box_rows) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return false;
  if (plane_stride <= 0) plane_stride = ld;   // never stepped over when it has one entry
  if (batch_stride <= 0) batch_stride = ld;
  cuuint64_t gdim[4] = {(cuuint64_t)inner, (cuuint64_t)rows, 3, (cuuint64_t)batch};
  cuuint64_t gstr[3] = {(cuuint64_t)ld * 2, (cuuint64_t)plane_stride * 2,
                        (cuuint64_t)batch_stride * 2};
  cuuint32_t box[4] = {(cuuint32_t)box_inner, (cuuint32_t)box_rows, 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<__nv_bfloat16*>(base), gdim, gstr,
             box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
             CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

__global__ void __launch_bounds__(256)
split3_kernel(const float* __restrict__ X, int64_t ld, int64_t rows, int64_t cols,
              __nv_bfloat16* __restrict__ planes, int64_t ldp, int64_t plane_stride) {
  const int64_t q4 = cols >> 2;
  const int64_t total = rows * q4;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += stride) {
    const int64_t r = e / q4;
    const int64_t cq = e - r * q4;
    const float4 x = *reinterpret_cast<const float4*>(X + r * ld + 4 * cq);
    float o[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
    for (int pl = 0; pl < 3; ++pl) {
      __nv_bfloat16 hb[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        hb[k] = __float2bfloat16_rn(o[k]);
        o[k] -= __bfloat162float(hb[k]);
      }
      uint2 pk;
      pk.x = (uint32_t)__bfloat16_as_ushort(hb[0]) | ((uint32_t)__bfloat16_as_ushort(hb[1]) << 16);
      pk.y = (uint32_t)__bfloat16_as_ushort(hb[2]) | ((uint32_t)__bfloat16_as_ushort(hb[3]) << 16);
      *reinterpret_cast<uint2*>(planes + (int64_t)pl * plane_stride + r * ldp + 4 * cq) = pk;
    }
  }
}

}  // namespace

thanos_status_t tc_gemm_split3(const TcGemmArgs& a, cudaStream_t stream) {
  if (a.M <= 0 || a.N <= 0 || a.batch <= 0) return THANOS_OK;
  if (a.K <= 0 || !a.A || !a.B || (!a.D && !a.Dp)) return THANOS_ERR_INVALID_ARG;
  if (!aligned16(a.A) || !aligned16(a.B) || !aligned16(a.D) || !aligned16(a.Dp))
    return THANOS_ERR_ALIGNMENT;
  if (a.lda % 8 || a.ldb % 8 || a.a_plane % 8 || a.b_plane % 8 || a.a_batch % 8 || a.b_batch % 8)
    return THANOS_ERR_ALIGNMENT;
  if (a.D && (a.ldd % 4 || a.d_batch % 4)) return THANOS_ERR_ALIGNMENT;
  if (a.Dp && (a.ldp % 4 || a.dp_plane % 4 || a.dp_batch % 4)) return THANOS_ERR_ALIGNMENT;
  CUtensorMap mapA, mapB;
  if (!make_map(&mapA, a.A, a.K, a.M, a.lda, a.a_plane, a.batch, a.a_batch, 64, 128))
    return THANOS_ERR_CUDA;
  const bool okb = a.b_kmajor
                       ? make_map(&mapB, a.B, a.K, a.N, a.ldb, a.b_plane, a.batch, a.b_batch, 64, 128)
                       : make_map(&mapB, a.B, a.N, a.K, a.ldb, a.b_plane, a.batch, a.b_batch, 64, 64);
  if (!okb) return THANOS_ERR_CUDA;
  CUtensorMap mapD = mapA;  // placeholder when no fp32 output is requested
  if (a.D) {
    EncodeTiledFn enc = encode_fn();
    const int64_t dbs = a.d_batch > 0 ? a.d_batch : a.ldd;
    cuuint64_t gdim[3] = {(cuuint64_t)a.N, (cuuint64_t)a.M, (cuuint64_t)a.batch};
    cuuint64_t gstr[2] = {(cuuint64_t)a.ldd * 4, (cuuint64_t)dbs * 4};
    cuuint32_t box[3] = {32, 128, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    if (!enc || enc(&mapD, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, a.D, gdim, gstr, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return THANOS_ERR_CUDA;
  }
  Params p;
  p.D = a.D;
  p.Dp = a.Dp;
  p.ldd = a.ldd;
  p.d_batch = a.d_batch;
  p.ldp = a.ldp;
  p.dp_plane = a.dp_plane;
  p.dp_batch = a.dp_batch;
  p.status = a.status;
  p.M = a.M;
  p.N = a.N;
  p.K = a.K;
  p.batch = a.batch;
  p.tiles_m = (a.M + TM - 1) / TM;
  p.tiles_n = (a.N + TN - 1) / TN;
  p.b_kmajor = a.b_kmajor;
  p.accumulate = a.accumulate;
  p.upper_only = a.upper_only;
  p.a_upper = a.a_upper;
  p.b_upper = a.b_upper;
  p.alpha = a.alpha;
  const long long tiles = (long long)p.tiles_m * p.tiles_n * p.batch;
  if (tiles > (1ll << 30)) return THANOS_ERR_SHAPE;
  // Large products go to CTA pairs (256 x 256 tiles): products with K >= 256 once they fill the
  // pairs at least twice over, rank-128 updates (bound by moving D, not by their operands) only
  // when they are an order of magnitude larger; never when the ragged edges of the wider tiles
  // would waste more than a fifth of the pairs' work.
  {
    const int pm = (a.M + PTM - 1) / PTM, pn = (a.N + PTN - 1) / PTN;
    const double used = ((double)a.M * (double)a.N) / ((double)pm * PTM * (double)pn * PTN);
    long long ptiles = (long long)pm * pn * p.batch;
    if (a.upper_only) ptiles = (ptiles + 1) / 2;
    int GP = 0;
    if (a.M >= PTM && a.N >= PTN && used >= 0.8) {
      // the shared-memory limit of the kernel has to be raised before its occupancy is asked for
      static std::atomic<unsigned long long> done{0};
      THANOS_CUDA(ensure_max_dyn_smem(tc_gemm_pair_kernel, (int)SMEM_BYTES, done));
      GP = max_active_gemm_pairs();
    }
    if (GP >= 8 && ptiles >= 2ll * GP && (a.K >= 256 || ptiles >= 12ll * GP)) {
      p.tiles_m = pm;
      p.tiles_n = pn;
      const long long all = (long long)pm * pn * p.batch;
      const int pairs = (int)(all < GP ? all : GP);
      tc_gemm_pair_kernel<<<2 * pairs, NTHREADS, SMEM_BYTES, stream>>>(mapA, mapB, mapD, p);
      THANOS_CHECK_LAUNCH();
      return THANOS_OK;
    }
  }
  const int G = sm_count();
  const int grid = (int)(tiles < G ? tiles : G);
  {
    static std::atomic<unsigned long long> done{0};
    THANOS_CUDA(ensure_max_dyn_smem(tc_gemm_kernel, (int)SMEM_BYTES, done));
  }
  tc_gemm_kernel<<<grid, NTHREADS, SMEM_BYTES, stream>>>(mapA, mapB, mapD, p);
  THANOS_CHECK_LAUNCH();
  return THANOS_OK;
}

thanos_status_t split3_planes(const float* X, int64_t ld, int64_t rows, int64_t cols,
                              __nv_bfloat16* planes, int64_t ldp, int64_t plane_stride,
                              cudaStream_t stream) {
  if (rows <= 0 || cols <= 0) return THANOS_OK;
  if (cols % 4 || ld % 4 || ldp % 4 || plane_stride % 4) return THANOS_ERR_ALIGNMENT;
  int64_t blocks = ceil_div(rows * (cols / 4), 256);
  if (blocks > NUM_SMS * 16) blocks = NUM_SMS * 16;
  split3_kernel<<<(unsigned)blocks, 256, 0, stream>>>(X, ld, rows, cols, planes, ldp, plane_stride);
  THANOS_CHECK_LAUNCH();
  return THANOS_OK;
}

}  // namespace thanos
