// Register-tiled fp32 GEMM tile on the plain ALUs.  Used where the contraction is small,
// skinny or must be fp32-exact (factorisation panels, per-block inverse rows); the large
// contractions have tensor-core kernels of their own.
#pragma once

#include "common.cuh"

namespace thanos {

// acc(i, j) += sum_{k in [kbeg, kend)} A(m, k) * B(k, n) for the BM x BN tile at (m0, n0).
//   TRANSA = false: A(m, k) = A[m * lda + k]     true: A(m, k) = A[k * lda + m]
//   TRANSB = false: B(k, n) = B[k * ldb + n]     true: B(k, n) = B[n * ldb + k]
// Out-of-range rows / columns / k read as zero, so any M, N, K works.
// A thread owns TM x TN outputs split into 4-wide chunks strided across the tile, which keeps
// the shared-memory fragment loads conflict-free.
template <int BM, int BN, int BK, int TM, int TN, bool TRANSA, bool TRANSB, typename TA,
          typename TB>
struct SimtGemm {
  static_assert(TM % 4 == 0 && TN % 4 == 0, "fragments are built from 4-wide chunks");
  static constexpr int TX = BN / TN;
  static constexpr int TY = BM / TM;
  static constexpr int THREADS = TX * TY;
  static constexpr int LDA_S = BM + 4;
  static constexpr int LDB_S = BN + 4;
  static constexpr int SMEM_FLOATS = BK * (LDA_S + LDB_S);
  static constexpr int CM = TM / 4;  // chunks per thread along m
  static constexpr int CN = TN / 4;

  __device__ static __forceinline__ int row_of(int ty, int i) {
    return (i / 4) * (BM / CM) + ty * 4 + (i % 4);
  }
  __device__ static __forceinline__ int col_of(int tx, int j) {
    return (j / 4) * (BN / CN) + tx * 4 + (j % 4);
  }

  __device__ static void run(const TA* __restrict__ A, int64_t lda, const TB* __restrict__ B,
                             int64_t ldb, int M, int N, int m0, int n0, int kbeg, int kend,
                             float (&acc)[TM][TN], float* smem) {
    float* As = smem;
    float* Bs = smem + BK * LDA_S;
    const int tid = threadIdx.x;
    const int tx = tid % TX;
    const int ty = tid / TX;

    for (int k0 = kbeg; k0 < kend; k0 += BK) {
      // ---- stage A tile as As[k][m]
      if (TRANSA) {
        for (int e = tid; e < BK * BM; e += THREADS) {
          int m = e % BM, k = e / BM;
          int gm = m0 + m, gk = k0 + k;
          float v = 0.f;
          if (gm < M && gk < kend) v = to_float(A[(int64_t)gk * lda + gm]);
          As[k * LDA_S + m] = v;
        }
      } else {
        for (int e = tid; e < BK * BM; e += THREADS) {
          int k = e % BK, m = e / BK;
          int gm = m0 + m, gk = k0 + k;
          float v = 0.f;
          if (gm < M && gk < kend) v = to_float(A[(int64_t)gm * lda + gk]);
          As[k * LDA_S + m] = v;
        }
      }
      // ---- stage B tile as Bs[k][n]
      if (!TRANSB) {
        for (int e = tid; e < BK * BN; e += THREADS) {
          int n = e % BN, k = e / BN;
          int gn = n0 + n, gk = k0 + k;
          float v = 0.f;
          if (gn < N && gk < kend) v = to_float(B[(int64_t)gk * ldb + gn]);
          Bs[k * LDB_S + n] = v;
        }
      } else {
        for (int e = tid; e < BK * BN; e += THREADS) {
          int k = e % BK, n = e / BK;
          int gn = n0 + n, gk = k0 + k;
          float v = 0.f;
          if (gn < N && gk < kend) v = to_float(B[(int64_t)gn * ldb + gk]);
          Bs[k * LDB_S + n] = v;
        }
      }
      __syncthreads();
#pragma unroll
      for (int k = 0; k < BK; ++k) {
        float a[TM], bfr[TN];
#pragma unroll
        for (int ci = 0; ci < CM; ++ci) {
          float4 v = *reinterpret_cast<const float4*>(&As[k * LDA_S + ci * (BM / CM) + ty * 4]);
          a[ci * 4 + 0] = v.x; a[ci * 4 + 1] = v.y; a[ci * 4 + 2] = v.z; a[ci * 4 + 3] = v.w;
        }
#pragma unroll
        for (int cj = 0; cj < CN; ++cj) {
          float4 v = *reinterpret_cast<const float4*>(&Bs[k * LDB_S + cj * (BN / CN) + tx * 4]);
          bfr[cj * 4 + 0] = v.x; bfr[cj * 4 + 1] = v.y; bfr[cj * 4 + 2] = v.z; bfr[cj * 4 + 3] = v.w;
        }
#pragma unroll
        for (int i = 0; i < TM; ++i)
#pragma unroll
          for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(a[i], bfr[j], acc[i][j]);
      }
      __syncthreads();
    }
  }
};

}  // namespace thanos
