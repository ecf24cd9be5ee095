// fp32-accurate GEMM on the bf16 tensor cores.
//
// Every fp32 operand is held as three bf16 planes x = h + m + l (24 significant bits); the six
// plane products hh, hm, mh, hl, lh, mm are accumulated in fp32 in tensor memory, the dropped
// ones are below 2^-24 relative.  Used for the dense contractions of the sweep (Eq. 8 for all
// rows of a block at once: W[:, j2:] += delta P2) and of the factorisation.
#pragma once

#include "common.cuh"

namespace thanos {

struct TcGemmArgs {
  // D[z][m, n] = (accumulate ? D[z][m, n] : 0) + alpha * sum_k A[z][m, k] * Bop[z][k, n]
  float* D = nullptr;            // fp32 [M, N], leading dimension ldd (may be null if Dp is set)
  int64_t ldd = 0;
  int64_t d_batch = 0;           // element stride between batch entries
  __nv_bfloat16* Dp = nullptr;   // optional: the result also as three bf16 planes
  int64_t ldp = 0;
  int64_t dp_plane = 0;
  int64_t dp_batch = 0;
  const __nv_bfloat16* A = nullptr;  // planes [3][M, K], K contiguous
  int64_t lda = 0;
  int64_t a_plane = 0;
  int64_t a_batch = 0;
  const __nv_bfloat16* B = nullptr;  // planes: b_kmajor ? [3][N, K] (K contiguous) : [3][K, N]
  int64_t ldb = 0;
  int64_t b_plane = 0;
  int64_t b_batch = 0;
  int b_kmajor = 1;
  int M = 0, N = 0, K = 0, batch = 1;
  float alpha = 1.f;
  int accumulate = 0;
  int upper_only = 0;            // skip tiles that lie strictly below the diagonal (n0 + 127 < m0)
  int a_upper = 0;               // A[m, k] = 0 for k < m: a tile starts its k loop at its first row
  int b_upper = 0;               // Bop[k, n] = 0 for k > n: a tile ends its k loop at its last column
  int32_t* status = nullptr;     // device int32: THANOS_ERR_TIMEOUT if a bounded wait ran out
};

// Pointers 16-byte aligned; lda, ldb, ldp and the plane / batch strides multiples of 8 elements.
thanos_status_t tc_gemm_split3(const TcGemmArgs& args, cudaStream_t stream);

// x -> three bf16 planes (h, m, l) of an fp32 matrix [rows, cols] (leading dimension ld);
// planes [3][rows, ldp].
thanos_status_t split3_planes(const float* X, int64_t ld, int64_t rows, int64_t cols,
                              __nv_bfloat16* planes, int64_t ldp, int64_t plane_stride,
                              cudaStream_t stream);

}  // namespace thanos
