/*
 * thanos.h -- C ABI of the B200 (sm_100a) library for the per-layer hot path of the Thanos
 * block-wise pruning method (arXiv 2504.05346).
 *
 * Notation follows the paper's notation table: a linear layer has weights W (c x b; c output
 * features = rows, b input features = columns), calibration inputs X (b x a; a tokens), the
 * Hessian H = 2 X X^T (b x b), block width B, sparsity ratio p, and a mask M with
 * M_ij = 1 meaning "weight W_ij is removed" (Section 2.1).
 *
 * Conventions shared by every call
 *  - All data pointers are DEVICE pointers unless the argument is documented as "host".
 *  - The caller owns every buffer.  The library allocates no device memory and keeps no
 *    global state between calls (except the entry point documented otherwise at the end of
 *    this header); scratch space is the caller-provided `workspace` whose minimum size
 *    comes from thanos_workspace_bytes().
 *  - Matrices are row-major and dense (leading dimension = number of columns) unless a
 *    leading dimension argument is present.
 *  - Calls are asynchronous: work is enqueued on `stream` (a cudaStream_t passed as
 *    void*; NULL is the legacy default stream) and the call returns without waiting.
 *  - Errors detectable on the host (null pointers, bad shapes, misalignment, workspace too
 *    small) are returned immediately and nothing is launched.  Conditions only the device
 *    can see (a non-positive Cholesky pivot, a bounded wait that ran out) are written to a
 *    status word in device memory (first error wins); the caller reads it after
 *    synchronising the stream.  Outputs are unspecified after an error.
 *  - Every pointer must be 16-byte aligned.
 */
#ifndef THANOS_H_
#define THANOS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  THANOS_OK = 0,
  THANOS_ERR_INVALID_ARG = 1, /* null pointer, value out of range                         */
  THANOS_ERR_SHAPE = 2,       /* a dimension violates a documented constraint              */
  THANOS_ERR_DTYPE = 3,       /* unknown thanos_dtype_t                                    */
  THANOS_ERR_ALIGNMENT = 4,   /* pointer or leading dimension not aligned as documented    */
  THANOS_ERR_WORKSPACE = 5,   /* workspace missing or smaller than thanos_workspace_bytes */
  THANOS_ERR_NOT_SPD = 6,     /* a Cholesky pivot was <= 0 or not finite (device status)   */
  THANOS_ERR_TIMEOUT = 7,     /* a bounded device-side wait expired (device status)        */
  THANOS_ERR_CUDA = 8         /* a CUDA runtime / driver call failed                       */
} thanos_status_t;

typedef enum { THANOS_F32 = 0, THANOS_BF16 = 1 } thanos_dtype_t;
typedef enum { THANOS_UNSTRUCTURED = 0, THANOS_NM = 1 } thanos_mode_t;

/* Which call a workspace query refers to. */
typedef enum {
  THANOS_WS_HESSIAN = 0,
  THANOS_WS_PREPARE = 1,
  THANOS_WS_PRUNE = 2,
  THANOS_WS_HOST_LAYER = 3,
  THANOS_WS_PRUNE_OUTLIERS = 4
} thanos_ws_which_t;

/* Per-call statistics and device-side status of thanos_prune_layer / thanos_prune_block,
 * written to device memory (64 bytes). */
typedef struct {
  int32_t status;       /* thanos_status_t of the first device-detected error, 0 if none  */
  int32_t err_index;    /* row (solve) or column (factorisation) where it was detected    */
  int64_t n_pruned;     /* number of mask entries set to 1 so far                          */
  int64_t r_left;       /* unstructured: removals still to place after the last block run */
  int32_t max_s;        /* largest per-row system size s seen                              */
  int32_t n_blocks;     /* column blocks processed                                         */
  int64_t n_tied;       /* unstructured: entries whose metric equals a block threshold
                           bit-for-bit but which the (row, column) tie-break left unpruned */
  uint32_t last_threshold_bits; /* fp32 bit pattern of the last block's threshold metric  */
  int32_t select_misses; /* unstructured: blocks whose threshold fell outside the bracket around
                            the previous block's (they take the four-pass route)              */
  int32_t select_rescans; /* unstructured: blocks whose bracket held more keys than the copy-out
                             buffers take (one CTA's share or the whole list), so that the
                             refining pass read the residual a second time                     */
  int32_t reserved[3];
} thanos_stats_t;

/*
 * Hessian accumulation: H += 2 * X_chunk^T X_chunk   (Section 3.2: H = 2 X X^T; summing over
 * calibration chunks is the un-averaged d-sample Hessian of Appendix A.4).
 *
 *  H       device, fp32 [b, b], full symmetric storage; the caller zeroes it before the first
 *          chunk.  Updated in place.  H[i][j] and H[j][i] receive the same addends, but in an
 *          unspecified order, so they may differ in the last bits; this library's own
 *          consumers read the upper triangle only.
 *  X       device, [n_tok, b] tokens-major (the transpose of the paper's X), element type
 *          `xdtype`, leading dimension `ldx` elements (ldx >= b, ldx % 8 == 0).
 *  b % 8 == 0, n_tok >= 0 (0 is a no-op).
 *  workspace: thanos_workspace_bytes(THANOS_WS_HESSIAN, 0, b, 0, xdtype) bytes.  Its first int32
 *          is this call's device status word: cleared when the call starts, set to
 *          THANOS_ERR_TIMEOUT if a bounded wait inside the tensor-core kernel ran out.
 * May be called any number of times; the order of floating-point summation across a call's
 * internal token slices is not fixed, so results can differ in the last bits between runs.
 */
thanos_status_t thanos_hessian_accumulate(float* H, int64_t b, const void* X,
                                          thanos_dtype_t xdtype, int64_t n_tok, int64_t ldx,
                                          void* workspace, size_t ws_bytes, void* stream);

/*
 * thanos_hessian_accumulate with a fixed order of floating-point summation (Section 3.2, as
 * above): a call is not split into concurrent token slices, so every entry of H receives exactly
 * one addend per call and the result -- hence the factor, the masks and the pruned weights that
 * follow from it -- is the same bit for bit from run to run for the same sequence of calls.
 * Same arguments and workspace.  A call with few tokens on a wide layer fills fewer SMs than the
 * unordered call would (its last wave of tiles can be up to half empty); calls of 16384 tokens
 * and more lose a few per cent.
 */
thanos_status_t thanos_hessian_accumulate_ordered(float* H, int64_t b, const void* X,
                                                  thanos_dtype_t xdtype, int64_t n_tok, int64_t ldx,
                                                  void* workspace, size_t ws_bytes, void* stream);

/*
 * Factor the damped Hessian so that the inverse of every trailing block is available
 * (Algorithm 1, last line of the block loop: the Hessian is restricted to the unseen columns
 * and re-inverted for every block; Appendix F.7 counts that as O(b^4 / B)).  This call
 * replaces all those inversions by one factorisation:
 *
 *   H_d = H + damp_rel * mean(diag H) * I          (damping as in Algorithm 5, line 3)
 *   factor = upper-triangular U with U^T U = H_d^{-1}; then for every j
 *   inv(H_d[j:, j:]) = U[j:, j:]^T U[j:, j:].
 *   xnorm[j] = sqrt(H_jj / 2) = ||X_j:||_2 from the UNDAMPED diagonal (metric of Eq. 4).
 *
 *  H        device, fp32 [b, b], read only (only the upper triangle is read).
 *  factor   device, fp32 [b, b]; entries below the diagonal are written as 0.
 *  xnorm    device, fp32 [b].
 *  status_dev device int32[2]: {thanos_status_t, failing column}; the caller zeroes it.
 *  workspace: thanos_workspace_bytes(THANOS_WS_PREPARE, 0, b, 0, THANOS_F32) bytes.
 * damp_rel >= 0; with damp_rel = 0 a singular H is reported as THANOS_ERR_NOT_SPD.
 */
thanos_status_t thanos_prepare_inverse(const float* H, int64_t b, float damp_rel, float* factor,
                                       float* xnorm, void* workspace, size_t ws_bytes,
                                       int32_t* status_dev, void* stream);

/*
 * Prune one layer: the block sweep of Algorithm 1 (mode THANOS_UNSTRUCTURED) or of
 * Algorithm 4 with alpha = 0 (mode THANOS_NM).  For each block of B columns, left to right:
 * metric |W_ij| * xnorm_j on the current weights (Section 4.2), block mask (Eq. psi over the
 * whole residual with running budget r = floor(p c b), or the n smallest of every aligned
 * group of m columns per row), per-row system lambda-hat R-hat = u and update
 * W_{i, j1:b} <- w - u R-hat^{-1} R (Eqs. 5-8), removed entries set to exact 0.
 *
 *  W_in     device [c, b], element type wdtype.
 *  W_out    device [c, b], same type; may alias W_in.
 *  mask_out device uint8 [c, b]; 1 = removed.
 *  factor, xnorm: outputs of thanos_prepare_inverse for this layer's input.
 *  mode UNSTRUCTURED: 0 <= p < 1 (n, m ignored).  Metric ties are broken by (row, column)
 *  ascending.  mode NM: 0 < n < m <= 32, B % m == 0, b % m == 0; n weights are REMOVED per
 *  group; ties by column ascending.
 *  1 <= B <= 512, B % 8 == 0, b % 8 == 0.  A row solves a system of min(|q|, |k|) <= B / 2
 *  unknowns (direct or complement form), so every admissible B is supported in both modes.
 *  stats_dev device thanos_stats_t, zeroed by this call.
 *  workspace: thanos_workspace_bytes(THANOS_WS_PRUNE, c, b, B, wdtype) bytes.
 */
thanos_status_t thanos_prune_layer(const void* W_in, void* W_out, uint8_t* mask_out,
                                   thanos_dtype_t wdtype, int64_t c, int64_t b,
                                   const float* factor, const float* xnorm, thanos_mode_t mode,
                                   double p, int32_t n, int32_t m, int32_t B, void* workspace,
                                   size_t ws_bytes, thanos_stats_t* stats_dev, void* stream);

/*
 * n:m sweep with outlier rows (Algorithm 4 with alpha > 0; outlier rows are defined in
 * Section 4.7): h_i = ||W_i X||_2^2 = 1/2 W_i H W_i^T is the loss of removing row i entirely; the
 * ceil(alpha c) rows with the largest h_i are left untouched (no entry removed, no update), every
 * other row is pruned exactly as by thanos_prune_layer in mode THANOS_NM.  The listing moves the
 * outlier rows last by a row permutation and undoes it at the end; rows are independent in n:m
 * mode, so this call skips them in place instead.  Equal losses are ordered by row index (the
 * higher index counts as the larger loss).
 *
 *  H        device fp32 [b, b], the UNDAMPED Hessian the factor was made from (full storage).
 *  alpha    0 <= alpha < 1; c - ceil(alpha c) rows are pruned.
 *  row_outlier_out  device uint8 [c] or NULL: 1 for the outlier rows.
 *  workspace: thanos_workspace_bytes(THANOS_WS_PRUNE_OUTLIERS, c, b, B, wdtype) bytes.
 * Everything else as in thanos_prune_layer.
 */
thanos_status_t thanos_prune_layer_outliers(const void* W_in, void* W_out, uint8_t* mask_out,
                                            thanos_dtype_t wdtype, int64_t c, int64_t b,
                                            const float* factor, const float* xnorm,
                                            const float* H, int32_t n, int32_t m, int32_t B,
                                            double alpha, uint8_t* row_outlier_out,
                                            void* workspace, size_t ws_bytes,
                                            thanos_stats_t* stats_dev, void* stream);

/*
 * Structured pruning (Algorithm 2, Section 4.7): whole columns are removed.  With
 * s = ceil(p b / (1 - alpha)), the ceil(alpha c) rows with the largest h_i (as in
 * thanos_prune_layer_outliers) are left untouched; over the other rows the s columns with the
 * smallest v_j = ||W_{rows, j}||_2^2 ||X_j||_2^2 form q (equal losses: the lower column first), and
 * every pruned row gets the multi-weight update of Eq. 8 with this same q,
 *     W <- W - W[:, q] inv(Hinv[q, q]) Hinv[q, :],   W[:, q] <- 0   (Hinv = inverse damped Hessian).
 * The listing permutes columns and rows to bring q and the pruned rows first and undoes both at
 * the end; this call gathers by index instead, which is the same arithmetic.
 *
 *  W_in, W_out   device [c, b] of wdtype, row-major, may alias.
 *  col_removed_out  device uint8 [b] or NULL: 1 for the removed columns.
 *  row_outlier_out  device uint8 [c] or NULL: 1 for the outlier rows.
 *  factor, xnorm    from thanos_prepare_inverse.
 *  H        device fp32 [b, b], the undamped Hessian; may be NULL when alpha == 0.
 *  p        0 <= p < 1, alpha 0 <= alpha < 1, and s < b, else THANOS_ERR_INVALID_ARG.
 *  b % 8 == 0, 8 <= b <= 65536, 1 <= c <= 2^24.
 *  stats_dev  device thanos_stats_t, written by this call: n_pruned = s (c - ceil(alpha c)),
 *           max_s = s, status THANOS_ERR_NOT_SPD if Hinv[q, q] is not positive definite in fp32.
 *  workspace: thanos_structured_workspace_bytes(c, b, p, alpha, wdtype) bytes.
 * Asynchronous on stream; no allocation.
 */
thanos_status_t thanos_prune_layer_structured(const void* W_in, void* W_out,
                                              uint8_t* col_removed_out, uint8_t* row_outlier_out,
                                              thanos_dtype_t wdtype, int64_t c, int64_t b,
                                              const float* factor, const float* xnorm,
                                              const float* H, double p, double alpha,
                                              void* workspace, size_t ws_bytes,
                                              thanos_stats_t* stats_dev, void* stream);

/* Workspace of thanos_prune_layer_structured; 0 if the arguments are not accepted. */
size_t thanos_structured_workspace_bytes(int64_t c, int64_t b, double p, double alpha,
                                         thanos_dtype_t dtype);

/*
 * One block step of the sweep from a caller-supplied state (the body of the block loop of
 * Algorithm 1 / Algorithm 4), for step-by-step checking against a reference.
 *
 *  Wc       device fp32 [c, b] working weights, updated in place for columns >= j1.
 *  mask     device uint8 [c, b]; columns [j1, min(b, j1+B)) are written.
 *  r_dev    device int64: removals still to place (unstructured); read and decremented by the
 *           number of entries this block removed.  Ignored in NM mode (may be NULL).
 *  stats_dev is accumulated into, not zeroed.  When it carries the statistics of the previous
 *           block step of the same sweep (n_blocks > 0), the unstructured threshold search starts
 *           from the bracket around last_threshold_bits (wide once select_misses > 0), exactly as
 *           inside thanos_prune_layer; with a zeroed stats_dev it starts from scratch (four radix
 *           passes).  Both routes give the same exact threshold.
 *  j1 % B == 0.  Same workspace as thanos_prune_layer.
 */
thanos_status_t thanos_prune_block(float* Wc, uint8_t* mask, int64_t c, int64_t b,
                                   const float* factor, const float* xnorm, thanos_mode_t mode,
                                   int32_t n, int32_t m, int32_t B, int64_t j1, int64_t* r_dev,
                                   void* workspace, size_t ws_bytes, thanos_stats_t* stats_dev,
                                   void* stream);

/*
 * The whole path for one layer from HOST buffers: copies X (in token chunks) and W to the
 * device, runs thanos_hessian_accumulate, thanos_prepare_inverse and thanos_prune_layer, and
 * copies W_pruned, the mask and the statistics back.  Synchronises `stream` before returning.
 *
 *  W_in_host, X_host, W_out_host, mask_out_host, stats_host: HOST pointers (pinned memory
 *  gives the best copy rate; pageable works).  X_host is [a, b] tokens-major.
 *  arena: DEVICE scratch of thanos_workspace_bytes(THANOS_WS_HOST_LAYER, c, b, B, dtype) bytes
 *  holding H, the factor, the staged inputs and the per-call workspaces.
 *  If reuse_factor != 0 the Hessian and factor left in `arena` by the previous call with the
 *  same b are reused and X_host is not read (layers that share an input, e.g. q/k/v).
 *  Unlike the device-pointer calls this one owns short-lived runtime objects: for the duration of
 *  a call that reads X_host it creates one copy stream and five events (so that the copy of a
 *  token chunk overlaps the accumulation of the previous one) and destroys them before returning;
 *  it allocates no memory.  stats_host->status also reports a bounded wait that ran out inside the
 *  Hessian accumulation (err_index -1) and a failed factorisation (err_index = column).
 */
thanos_status_t thanos_prune_layer_host(const void* W_in_host, const void* X_host,
                                        void* W_out_host, uint8_t* mask_out_host,
                                        thanos_dtype_t dtype, int64_t c, int64_t b, int64_t a,
                                        float damp_rel, thanos_mode_t mode, double p, int32_t n,
                                        int32_t m, int32_t B, int32_t reuse_factor, void* arena,
                                        size_t arena_bytes, thanos_stats_t* stats_host,
                                        void* stream);

/*
 * Variant of thanos_prune_layer for callers that cannot provide a workspace.  The paper has no
 * counterpart of this call; it computes exactly what thanos_prune_layer computes.
 *
 * Who needs it: code that runs where device memory can no longer be obtained -- a plugin
 * inside a serving process whose allocator already owns the whole GPU, a step of a pipeline
 * that must not call cudaMalloc because that call synchronises the device and would stall
 * the other streams, or a host that forbids allocation after start-up.  Such a caller has its
 * weights, the factor and the outputs, but no spare buffer to pass as `workspace`.
 *
 * The sweep's scratch is a fixed 4 MiB array that is part of the library's device image
 * (every GPU that loads the library holds it until the process exits).  The call allocates
 * nothing and frees nothing.  A layer fits when
 *     thanos_workspace_bytes(THANOS_WS_PRUNE, c, b, B, wdtype) <= 4 MiB
 * (for example 512 x 512 fp32 or 256 x 512 bf16 with B = 128); anything larger
 * is refused with THANOS_ERR_WORKSPACE before any work is enqueued.
 *
 * The first call on a device looks up the device address of that array (once per device, with
 * the device current); make this first call before starting any stream capture.  All calls
 * on a device share the one array: the call clears the parts that must start from zero, so
 * leftovers of an earlier call are harmless, but two calls that overlap on the GPU (different
 * streams, or different host threads) race on it -- serialise them.
 *
 * The array that is used is the current device's: make the device that holds W_in current
 * before the call (weights on another device are refused with THANOS_ERR_INVALID_ARG).
 *
 * Arguments, layouts, results and device-side error reporting are those of
 * thanos_prune_layer, minus `workspace` and `ws_bytes`.
 */
thanos_status_t thanos_prune_layer_noalloc(const void* W_in, void* W_out, uint8_t* mask_out,
                                           thanos_dtype_t wdtype, int64_t c, int64_t b,
                                           const float* factor, const float* xnorm,
                                           thanos_mode_t mode, double p, int32_t n, int32_t m,
                                           int32_t B, thanos_stats_t* stats_dev, void* stream);

/*
 * Dense product on the tensor cores with fp32 accuracy:
 *     D = (accumulate ? D : 0) + alpha * A * op(B)
 * This is the contraction behind Eq. 8 applied to every row of a block at once (the change of the
 * columns right of a block is delta times a matrix that depends only on the Hessian), exposed
 * so that it can be checked and timed on its own.  Every fp32 operand is split into three bf16
 * planes and six plane products are accumulated in fp32, so the result agrees with an fp32
 * product to a few units of 2^-24 of sum |a||b|.
 *
 *  D   device fp32 [M, N], leading dimension ldd (ldd % 4 == 0).
 *  A   device fp32 [M, K], leading dimension lda.
 *  B   device fp32; b_transposed != 0: [N, K] (op(B) = B^T), else [K, N]; leading dimension ldb.
 *  lda, ldb multiples of 4; K and the contiguous extent of B multiples of 4.
 *  workspace: thanos_dense_product_workspace(M, N, K) bytes; its first int32 is the device status
 *  word of the call (THANOS_ERR_TIMEOUT if a bounded wait ran out).
 */
thanos_status_t thanos_dense_product(float* D, int64_t ldd, const float* A, int64_t lda,
                                     const float* B, int64_t ldb, int32_t b_transposed, int64_t M,
                                     int64_t N, int64_t K, float alpha, int32_t accumulate,
                                     void* workspace, size_t ws_bytes, void* stream);
size_t thanos_dense_product_workspace(int64_t M, int64_t N, int64_t K);

/*
 * Measurement aid (the paper has no counterpart): launches `ctas` CTAs of 256 threads that each
 * run 16 independent chains of 4 * iters dependent fp32 FMAs and store one float per thread to
 * `out` (device, at least ctas * 256 floats).  *flop_out (host, may be NULL) receives the
 * floating-point operations of the launch, 2 per FMA.  Timed by the caller with events, this
 * gives the plain fp32 arithmetic peak of the device -- the roofline of the per-row solves.
 */
thanos_status_t thanos_fp32_fma_probe(float* out, int64_t out_elems, int32_t ctas, int32_t iters,
                                      double* flop_out, void* stream);

/* Minimum workspace in bytes for a call (see thanos_ws_which_t); 0 for unsupported shapes. */
size_t thanos_workspace_bytes(int32_t which, int64_t c, int64_t b, int32_t B, thanos_dtype_t dtype);

/* Static, NUL-terminated description of a status code. */
const char* thanos_status_string(thanos_status_t status);

/* Library version as major * 10000 + minor * 100 + patch. */
int32_t thanos_version(void);

/* Number of kernels this library has launched in the calling process since it was loaded
 * (host counter, for benchmarks that report launch counts). */
int64_t thanos_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* THANOS_H_ */
