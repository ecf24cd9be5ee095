"""Float64 CPU oracle for the Thanos per-layer pruning path.

TEST INFRASTRUCTURE ONLY.  This module is a plain, slow, step-by-step restatement of what
the paper defines, in NumPy float64.  It shares no code with the CUDA library and must never
be imported by the product path; only the test-suite, the smoke check and the benchmark's
CPU-baseline leg call it.

Orientation follows the paper's notation table: ``W`` is ``c x b`` (rows = output features,
columns = input features), ``X`` is ``b x a`` (row ``j`` holds input feature ``j`` over all
``a`` calibration tokens), ``H = 2 X X^T`` is ``b x b``, and a mask entry ``M_ij = 1`` means
"weight ``W_ij`` is removed" (Section 2.1).

Readings taken where the paper is silent or inconsistent (each is a convention of this
build, not something the paper fixes):

* block loop: 0-based ``j1 = 0, B, 2B, ... < b`` and ``j2 = min(b, j1 + B)``; the listing's
  bounds mix 1- and 0-based indexing (Algorithm 1, block loop) -- the text says there are
  ``ceil(b / B)`` blocks (Section 4.3);
* ``r = floor(p c b)`` (constraint of Eq. 2; Algorithm 1 writes ``p c b``);
* damping ``H_d = H + damp_rel * mean(diag H) * I`` -- the Thanos listings have no damping,
  the SparseGPT listing adds ``lambda I`` (Algorithm 5); ``damp_rel = 0`` gives the listing;
* the metric norms ``||X_j:||_2`` come from the undamped data (Eq. psi is defined on X);
* ties in the metric are broken by (value, row, column) ascending; n:m groups by column;
* the inverse used in a block is that of the residual Hessian ``H_d[j1:, j1:]`` (Algorithm 1,
  Hessian-update line at the end of the block loop);
* n:m: ``n`` weights are REMOVED out of every aligned group of ``m`` columns, per row
  (Section 4.8: every group of ``m`` consecutive weights contains exactly ``n`` zeros);
* removed entries are set to exact zero after the update (constraint of Eq. 2).

parity unpinned: the tie-break rule, the damping convention and the use of undamped norms
are not fixed by the paper; everything else below is pinned by the tests in
``tests/test_oracle_*.py``.
"""

from __future__ import annotations

import math

import numpy as np

F64 = np.float64


# --------------------------------------------------------------------------------------
# Hessian (Section 3.2, H = 2 X X^T; Appendix B.2 derivation; d-sample sum, Appendix A.4)
# --------------------------------------------------------------------------------------
def hessian(X: np.ndarray) -> np.ndarray:
    """``H = 2 X X^T`` for ``X`` of shape ``b x a`` (Section 3.2, below Eq. 3)."""
    X = np.asarray(X, dtype=F64)
    return 2.0 * (X @ X.T)


def hessian_from_chunks(chunks) -> np.ndarray:
    """Sum of ``2 X^l X^l^T`` over calibration chunks ``X^l`` (``b x a_l``), un-averaged.

    Appendix A.4 averages over ``d`` samples; the scale is irrelevant to the ranking of the
    metric, to a relative damping and to ``R-hat^{-1} R``, and this build keeps the plain sum.
    """
    H = None
    for Xl in chunks:
        Hl = hessian(Xl)
        H = Hl if H is None else H + Hl
    return H


def feature_norms(H: np.ndarray) -> np.ndarray:
    """``||X_j:||_2 = sqrt(H_jj / 2)`` from the undamped Hessian (Eq. 4)."""
    return np.sqrt(np.diag(np.asarray(H, dtype=F64)) / 2.0)


def damped(H: np.ndarray, damp_rel: float) -> np.ndarray:
    """``H_d = H + lambda I`` with ``lambda = damp_rel * mean(diag H)`` (Algorithm 5, line 3)."""
    H = np.asarray(H, dtype=F64)
    lam = float(damp_rel) * float(np.mean(np.diag(H)))
    return H + lam * np.eye(H.shape[0], dtype=F64)


# --------------------------------------------------------------------------------------
# Metric, psi and phi (Section 4.2, Eq. psi, Section 4.5)
# --------------------------------------------------------------------------------------
def metric(W: np.ndarray, xnorm: np.ndarray) -> np.ndarray:
    """``S_ij = |W_ij| * ||X_j:||_2`` (Eq. 4 / Section 4.2)."""
    return np.abs(np.asarray(W, dtype=F64)) * np.asarray(xnorm, dtype=F64)[None, :]


def psi(W: np.ndarray, xnorm: np.ndarray, r: int) -> np.ndarray:
    """Mask of the ``r`` entries of ``W`` with the smallest metric (Eq. psi).

    Equal metric values are ordered by (row, column): a stable sort of the row-major
    flattening does exactly that.
    """
    S = metric(W, xnorm)
    order = np.argsort(S.ravel(), kind="stable")
    M = np.zeros(S.size, dtype=np.uint8)
    M[order[: int(r)]] = 1
    return M.reshape(S.shape)


def phi(x: np.ndarray) -> np.ndarray:
    """0-based, ascending indices of the non-zero entries of a mask row (Section 4.5).

    The paper's examples are 1-based: ``phi((1,0,0,1,1)) = (1,4,5)``.
    """
    return np.flatnonzero(np.asarray(x))


def nm_block_mask(Wblk: np.ndarray, xnorm_blk: np.ndarray, n: int, m: int) -> np.ndarray:
    """Per row and per group of ``m`` consecutive columns, mark the ``n`` smallest-metric
    entries (Algorithm 4, inner mask loop).  A ragged last group of ``g < m`` columns marks
    ``min(n, g)`` entries."""
    c, w = Wblk.shape
    S = metric(Wblk, xnorm_blk)
    M = np.zeros((c, w), dtype=np.uint8)
    for g0 in range(0, w, m):
        g1 = min(w, g0 + m)
        k = min(n, g1 - g0)
        for i in range(c):
            order = np.argsort(S[i, g0:g1], kind="stable")
            M[i, g0 + order[:k]] = 1
    return M


# --------------------------------------------------------------------------------------
# Optimal multi-weight update for one row (Section 4.1, Eqs. 5-8; Appendix C.1)
# --------------------------------------------------------------------------------------
def row_update(Hinv: np.ndarray, q: np.ndarray, w: np.ndarray):
    """Optimal change of one row ``w`` (length of ``Hinv``) that zeroes positions ``q``.

    ``R = Hinv[q, :]`` (Eq. 5), ``R-hat = R[:, q]`` (Eq. 6), ``u = w[q]`` (Eq. 7); the
    multipliers solve ``lambda-hat R-hat = u`` and the change is ``-lambda-hat R`` (Eq. 8).
    Returns ``(delta, lambda_hat)``.
    """
    q = np.asarray(q, dtype=np.int64)
    R = Hinv[q, :]
    Rhat = R[:, q]
    u = w[q]
    lam = np.linalg.solve(Rhat.T, u)  # row vector times matrix: lam @ Rhat = u
    return -(lam @ R), lam


def row_loss(Hinv: np.ndarray, H: np.ndarray, q: np.ndarray, w: np.ndarray) -> float:
    """``S = 1/2 u R-hat^{-1} R H R^T R-hat^{-T} u^T`` (Eq. 8, second part), evaluated literally."""
    q = np.asarray(q, dtype=np.int64)
    R = Hinv[q, :]
    Rhat = R[:, q]
    u = w[q]
    t = np.linalg.solve(Rhat.T, u)  # u Rhat^{-1}
    return 0.5 * float(t @ R @ H @ R.T @ t)


def padded_system(Hinv: np.ndarray, q: np.ndarray, w: np.ndarray, r_max: int):
    """The padded system of Appendix G.1: index vector filled up to ``r_max`` with the
    first index, ``u' = (u, 0)``, ``R-hat' = diag(R-hat, I)``.  Returns
    ``(padded_indices, lambda_prime)``."""
    q = np.asarray(q, dtype=np.int64)
    s = q.size
    idx = np.concatenate([q, np.zeros(r_max - s, dtype=np.int64)])
    Rhat = Hinv[np.ix_(q, q)]
    Rp = np.eye(r_max, dtype=F64)
    Rp[:s, :s] = Rhat
    up = np.zeros(r_max, dtype=F64)
    up[:s] = w[q]
    lam_p = np.linalg.solve(Rp.T, up)
    return idx, lam_p


# --------------------------------------------------------------------------------------
# Algorithm 1 (unstructured) and Algorithm 4 (n:m, alpha = 0): literal block sweeps
# --------------------------------------------------------------------------------------
def _sweep(W, H, xnorm, B, damp_rel, block_mask_fn, collect=None):
    """Common block loop of Algorithms 1 and 4.  ``block_mask_fn(Wc, j1, j2)`` returns the
    local block mask ``M`` (c x (j2-j1)) from the current weights."""
    W = np.asarray(W, dtype=F64)
    c, b = W.shape
    Hd = damped(H, damp_rel)
    Wc = W.copy()
    M = np.zeros((c, b), dtype=np.uint8)
    for j1 in range(0, b, B):
        j2 = min(b, j1 + B)
        Mb = block_mask_fn(Wc, j1, j2)
        # inverse of the residual Hessian: columns < j1 are final and no longer take part
        Hinv = np.linalg.inv(Hd[j1:, j1:])
        if collect is not None:
            collect.append({"j1": j1, "j2": j2, "W_before": Wc.copy(), "mask": Mb.copy(),
                            "loss": 0.0})
        for i in range(c):
            q = phi(Mb[i])
            if q.size == 0:
                continue
            w = Wc[i, j1:]
            delta, lam = row_update(Hinv, q, w)
            if collect is not None:
                collect[-1]["loss"] += 0.5 * float(lam @ w[q])  # 1/2 u Rhat^{-1} u^T
            Wc[i, j1:] = w + delta
            Wc[i, j1 + q] = 0.0
        M[:, j1:j2] = Mb
    return Wc, M


def thanos_unstructured(W, X, p, B, damp_rel=0.0, H=None, collect=None):
    """Algorithm 1: global residual mask with a running budget ``r``.

    Returns ``(W_pruned, M, H)``; ``H`` may be supplied (already ``2 X X^T``) to skip the
    Hessian.
    """
    W = np.asarray(W, dtype=F64)
    c, b = W.shape
    if H is None:
        H = hessian(X)
    xn = feature_norms(H)
    state = {"r": int(math.floor(p * c * b))}

    def block_mask(Wc, j1, j2):
        Mhat = psi(Wc[:, j1:], xn[j1:], state["r"])  # global residual mask
        Mb = Mhat[:, : j2 - j1]  # local block mask
        state["r"] -= int(Mb.sum())
        return Mb

    Wp, M = _sweep(W, H, xn, B, damp_rel, block_mask, collect)
    return Wp, M, H


def row_losses(W, X=None, H=None):
    """``h_i = ||W_i X||_2^2``: the loss of Eq. 1 when row ``i`` is removed entirely (definition
    of the outlier rows, Section 4.7).  From the Hessian it is ``1/2 W_i H W_i^T``."""
    W = np.asarray(W, dtype=F64)
    if X is not None:
        return np.sum((W @ np.asarray(X, dtype=F64)) ** 2, axis=1)
    return 0.5 * np.einsum("ij,jk,ik->i", W, np.asarray(H, dtype=F64), W)


def outlier_row_order(h, alpha):
    """Row permutation of Algorithm 4: rows in ascending order of ``h`` (stable: equal losses keep
    their row order), so the ``ceil(alpha c)`` outlier rows come last.  Returns
    ``(sigma, n_out)`` with ``sigma[k]`` = original index of the row at position ``k``.

    Reading: the section defining alpha fixes the number of outlier rows as ``ceil(alpha c)``; the
    listing's row loop runs to ``ceil(c (1 - alpha))``, which is one more row when ``alpha c`` is
    not an integer.  The count from the definition is used: ``c - ceil(alpha c)`` rows are pruned.
    """
    h = np.asarray(h, dtype=F64)
    c = h.shape[0]
    n_out = int(math.ceil(float(alpha) * c - 1e-12)) if alpha > 0 else 0
    sigma = np.argsort(h, kind="stable")
    return sigma, n_out


def thanos_nm(W, X, n, m, B, damp_rel=0.0, H=None, collect=None, alpha=0.0):
    """Algorithm 4.  ``alpha`` is the fraction of outlier rows: the ``ceil(alpha c)`` rows with the
    largest ``h_i = ||W_i X||^2`` are moved last by the row permutation ``Q`` and are not pruned;
    the inverse permutation restores the row order at the end."""
    W = np.asarray(W, dtype=F64)
    if B % m != 0:
        raise ValueError("block size B must be a multiple of m")
    if H is None:
        H = hessian(X)
    xn = feature_norms(H)
    c = W.shape[0]
    if alpha > 0:
        sigma, n_out = outlier_row_order(row_losses(W, H=H), alpha)
    else:
        sigma, n_out = np.arange(c), 0
    Wq = W[sigma]                      # W <- Q W
    n_pruned_rows = c - n_out

    def block_mask(Wc, j1, j2):
        Mb = nm_block_mask(Wc[:, j1:j2], xn[j1:j2], n, m)
        Mb[n_pruned_rows:] = 0         # the row loop of the listing stops before the outliers
        return Mb

    Wp, M = _sweep(Wq, H, xn, B, damp_rel, block_mask, collect)
    inv = np.empty(c, dtype=np.int64)
    inv[sigma] = np.arange(c)
    return Wp[inv], M[inv], H          # W <- Q^T W


# --------------------------------------------------------------------------------------
# Structured pruning (Algorithm 2): whole columns, one shared system for all rows
# --------------------------------------------------------------------------------------
def column_losses(W_rows, xnorm):
    """``v_j = ||W_{rows, j} (x) X_j||_F^2 = ||W_{rows, j}||^2 ||X_j||^2`` over the rows that are
    pruned (Eq. for the column loss, Section 4.7; ``xnorm_j = ||X_j||_2``)."""
    W_rows = np.asarray(W_rows, dtype=F64)
    return np.sum(W_rows ** 2, axis=0) * np.asarray(xnorm, dtype=F64) ** 2


def structured_column_count(p, b, alpha):
    """``s = ceil(p b / (1 - alpha))`` columns are removed (Algorithm 2, first line)."""
    return int(math.ceil(float(p) * b / (1.0 - float(alpha)) - 1e-12))


def thanos_structured(W, X, p, alpha=0.0, damp_rel=0.0, H=None):
    """Algorithm 2.  Rows are permuted so that the ``ceil(alpha c)`` outlier rows (largest
    ``h_i``) come last, columns so that the ``s`` columns with the smallest ``v_j`` come first;
    the pruned rows get ``W - W[:, :s] inv(Hinv[:s, :s]) Hinv[:s, :]`` (Eq. 8 with the same ``q``
    for every row) and exact zeros in the removed columns; the permutations are undone.
    Outlier rows are not changed at all.  Returns ``(W_pruned, removed_columns, outlier_rows, H)``
    with boolean index arrays in the original order.

    Readings: the listing writes the update as an assignment to ``W[:, 1:s]`` with a right-hand
    side of width ``b`` -- taken as the update of the whole (pruned) rows, as in Eq. 8; ``H^{-1}``
    is the inverse of the damped Hessian; ties in ``v_j`` keep the column order."""
    W = np.asarray(W, dtype=F64)
    c, b = W.shape
    if H is None:
        H = hessian(X)
    xn = feature_norms(H)
    s = structured_column_count(p, b, alpha)
    if not 0 <= s < b:
        raise ValueError("p / (1 - alpha) must leave at least one column")
    if alpha > 0:
        sigma_r, n_out = outlier_row_order(row_losses(W, H=H), alpha)
    else:
        sigma_r, n_out = np.arange(c), 0
    Wq = W[sigma_r]                                   # W' = Q W
    n_rows = c - n_out
    v = column_losses(Wq[:n_rows], xn)
    sigma_c = np.argsort(v, kind="stable")            # columns with the smallest loss first
    Wp = Wq[:, sigma_c]                               # W' P
    Hinv = np.linalg.inv(damped(H, damp_rel))[np.ix_(sigma_c, sigma_c)]
    if s > 0:
        lam = np.linalg.solve(Hinv[:s, :s].T, Wp[:n_rows, :s].T).T   # W[:, :s] inv(Hinv[:s,:s])
        Wp[:n_rows] = Wp[:n_rows] - lam @ Hinv[:s, :]
        Wp[:n_rows, :s] = 0.0
    inv_c = np.empty(b, dtype=np.int64)
    inv_c[sigma_c] = np.arange(b)
    inv_r = np.empty(c, dtype=np.int64)
    inv_r[sigma_r] = np.arange(c)
    out = Wp[:, inv_c][inv_r]
    removed = np.zeros(b, dtype=bool)
    removed[sigma_c[:s]] = True
    outl = np.zeros(c, dtype=bool)
    outl[sigma_r[n_rows:]] = True
    return out, removed, outl, H


def structured_update_rows(W_rows, removed, Hd):
    """Eq. 8 for given rows with a given set of removed columns ``q`` (boolean [b]):
    ``w - w_q inv(Hinv[q, q]) Hinv[q, :]`` and zeros at ``q`` -- the row update of Algorithm 2
    without its permutations, for checking sampled rows of a large layer."""
    W_rows = np.asarray(W_rows, dtype=F64)
    q = np.nonzero(np.asarray(removed, dtype=bool))[0]
    if q.size == 0:
        return W_rows.copy()
    Hinv = np.linalg.inv(np.asarray(Hd, dtype=F64))
    lam = np.linalg.solve(Hinv[np.ix_(q, q)].T, W_rows[:, q].T).T
    out = W_rows - lam @ Hinv[q, :]
    out[:, q] = 0.0
    return out


# --------------------------------------------------------------------------------------
# Faster float64 route for larger shapes: one factorisation instead of one inverse per block.
# Allowed only because tests show it equals the literal sweep to ~1e-10 on small shapes.
# --------------------------------------------------------------------------------------
def inverse_factor(Hd: np.ndarray) -> np.ndarray:
    """Upper-triangular ``U`` with ``U^T U = Hd^{-1}``.

    For every ``j``: ``inv(Hd[j:, j:]) = U[j:, j:]^T U[j:, j:]`` (Schur complement of the
    leading block of ``Hd^{-1}``), which replaces the per-block re-inversion of Algorithm 1.
    """
    Hinv = np.linalg.inv(np.asarray(Hd, dtype=F64))
    Hinv = 0.5 * (Hinv + Hinv.T)
    return np.linalg.cholesky(Hinv).T


def block_update_from_factor(Wc, Mb, U, j1, j2):
    """One block of the sweep (in place on ``Wc[:, j1:]``) with the residual inverse rows
    rebuilt from the factor ``U``: Eqs. 5-8 for every row, removed entries set to 0."""
    c = Wc.shape[0]
    Ubb = U[j1:j2, j1:j2]
    P = Ubb.T @ U[j1:j2, j1:]  # rows j1..j2 of inv(Hd[j1:, j1:])
    G = P[:, : j2 - j1]
    Lam = np.zeros((c, j2 - j1), dtype=F64)
    for i in range(c):
        q = phi(Mb[i])
        if q.size == 0:
            continue
        Lam[i, q] = np.linalg.solve(G[np.ix_(q, q)].T, Wc[i, j1 + q])
    Wc[:, j1:] -= Lam @ P
    blk = Wc[:, j1:j2]
    blk[Mb.astype(bool)] = 0.0


def _sweep_fast(W, H, xnorm, B, damp_rel, block_mask_fn):
    W = np.asarray(W, dtype=F64)
    c, b = W.shape
    U = inverse_factor(damped(H, damp_rel))
    Wc = W.copy()
    M = np.zeros((c, b), dtype=np.uint8)
    for j1 in range(0, b, B):
        j2 = min(b, j1 + B)
        Mb = block_mask_fn(Wc, j1, j2)
        block_update_from_factor(Wc, Mb, U, j1, j2)
        M[:, j1:j2] = Mb
    return Wc, M


def thanos_unstructured_fast(W, X, p, B, damp_rel=0.0, H=None):
    W = np.asarray(W, dtype=F64)
    c, b = W.shape
    if H is None:
        H = hessian(X)
    xn = feature_norms(H)
    state = {"r": int(math.floor(p * c * b))}

    def block_mask(Wc, j1, j2):
        Mhat = psi(Wc[:, j1:], xn[j1:], state["r"])
        Mb = Mhat[:, : j2 - j1]
        state["r"] -= int(Mb.sum())
        return Mb

    Wp, M = _sweep_fast(W, H, xn, B, damp_rel, block_mask)
    return Wp, M, H


def thanos_nm_fast(W, X, n, m, B, damp_rel=0.0, H=None):
    W = np.asarray(W, dtype=F64)
    if B % m != 0:
        raise ValueError("block size B must be a multiple of m")
    if H is None:
        H = hessian(X)
    xn = feature_norms(H)

    def block_mask(Wc, j1, j2):
        S = metric(Wc[:, j1:j2], xn[j1:j2])
        c, w = S.shape
        Mb = np.zeros((c, w), dtype=np.uint8)
        for g0 in range(0, w, m):
            g1 = min(w, g0 + m)
            k = min(n, g1 - g0)
            order = np.argsort(S[:, g0:g1], axis=1, kind="stable")[:, :k]
            np.put_along_axis(Mb[:, g0:g1], order, 1, axis=1)
        return Mb

    Wp, M = _sweep_fast(W, H, xn, B, damp_rel, block_mask)
    return Wp, M, H


# --------------------------------------------------------------------------------------
# Replay of the sweep for chosen rows under a GIVEN mask (rows are independent once the
# mask is fixed: Eq. "separated loss", Appendix A.3).  Used to check results at sizes where
# the full sweep is too slow for the CPU.
# --------------------------------------------------------------------------------------
def replay_rows(W_rows, M_rows, Hd, B):
    """Apply the block sweep's update (Eq. 8 per block) to the given rows with the given
    full-width mask rows.  ``Hd`` is the damped Hessian."""
    W_rows = np.asarray(W_rows, dtype=F64).copy()
    nrow, b = W_rows.shape
    U = inverse_factor(Hd)
    for j1 in range(0, b, B):
        j2 = min(b, j1 + B)
        Ubb = U[j1:j2, j1:j2]
        P = Ubb.T @ U[j1:j2, j1:]
        G = P[:, : j2 - j1]
        for i in range(nrow):
            q = phi(M_rows[i, j1:j2])
            if q.size == 0:
                continue
            lam = np.linalg.solve(G[np.ix_(q, q)].T, W_rows[i, j1 + q])
            W_rows[i, j1:] -= lam @ P[q, :]
            W_rows[i, j1 + q] = 0.0
    return W_rows


# --------------------------------------------------------------------------------------
# Objective (Eq. 1) and the magnitude baseline used for a sanity comparison
# --------------------------------------------------------------------------------------
def objective(W_hat, W, X) -> float:
    """``f(W_hat) = ||(W_hat - W) X||_F^2`` (Eq. 1)."""
    D = np.asarray(W_hat, dtype=F64) - np.asarray(W, dtype=F64)
    return float(np.sum((D @ np.asarray(X, dtype=F64)) ** 2))


def objective_H(W_hat, W, H) -> float:
    """Same objective through the Hessian: ``1/2 sum_i Delta_i H Delta_i^T``."""
    D = np.asarray(W_hat, dtype=F64) - np.asarray(W, dtype=F64)
    return 0.5 * float(np.sum((D @ np.asarray(H, dtype=F64)) * D))


def zero_without_update(W, M):
    """``W - M * W``: remove the masked weights and change nothing else (Algorithm 3, last line)."""
    return np.asarray(W, dtype=F64) * (1 - np.asarray(M, dtype=F64))
