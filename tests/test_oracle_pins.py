"""Pins for the float64 oracle: every check here compares the oracle with something other
than itself -- values printed in the paper, closed forms, brute force, or library routines
applied to the problem's plain definition."""

import math
import os

import numpy as np
import pytest

from oracle import thanos_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _read_sections(path):
    sec, cur = {}, None
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line[0].isalpha():
            cur = line
            sec[cur] = []
        else:
            sec[cur].append([float(t) for t in line.split()])
    return {k: np.array(v) for k, v in sec.items()}


def _rand_problem(rng, c, b, a, corr=0.5):
    X = rng.standard_normal((b, a))
    X = (np.eye(b) + corr * rng.standard_normal((b, b)) / math.sqrt(b)) @ X
    X[rng.integers(0, b)] *= 5.0
    W = rng.standard_normal((c, b)) * 0.02
    return W, X


# ---------------------------------------------------------------- values printed in the paper
def test_psi_worked_example_from_paper():
    g = _read_sections(os.path.join(GOLD, "psi_worked_example.txt"))
    W, X = g["W"], g["X"]
    H = O.hessian(X)
    xn = O.feature_norms(H)
    # norms are taken over the ROWS of X (per input feature): (5, 1)
    assert np.allclose(xn, [5.0, 1.0])
    assert np.array_equal(O.metric(W, xn), g["metric"])
    for r in (1, 2, 4):
        assert np.array_equal(O.psi(W, xn, r), g["psi %d" % r].astype(np.uint8)), r


def test_phi_examples_from_paper():
    for line in open(os.path.join(GOLD, "phi_examples.txt")):
        if line.startswith("#") or "->" not in line:
            continue
        lhs, rhs = line.split("->")
        x = np.array([int(t) for t in lhs.split()])
        want = np.array([int(t) for t in rhs.split()])
        assert np.array_equal(O.phi(x) + 1, want)  # the paper counts from 1


def test_padded_system_example_from_paper():
    rng = np.random.default_rng(5)
    b = 7
    A = rng.standard_normal((b, 3 * b))
    Hinv = np.linalg.inv(2 * A @ A.T)
    w = rng.standard_normal(b)
    q = np.array([1, 2, 5]) - 1
    idx, lam_p = O.padded_system(Hinv, q, w, r_max=5)
    assert np.array_equal(idx + 1, [1, 2, 5, 1, 1])
    _, lam = O.row_update(Hinv, q, w)
    assert np.allclose(lam_p[:3], lam, rtol=1e-12, atol=0)
    assert np.all(lam_p[3:] == 0.0)


# ---------------------------------------------------------------- Hessian
def test_hessian_matches_elementwise_definition():
    rng = np.random.default_rng(0)
    X = rng.standard_normal((5, 9))
    H = O.hessian(X)
    for i in range(5):
        for j in range(5):
            acc = 0.0
            for t in range(9):
                acc += X[i, t] * X[j, t]
            assert abs(H[i, j] - 2 * acc) < 1e-12
    assert np.array_equal(H, H.T)
    assert np.all(np.linalg.eigvalsh(H) > 0)


def test_hessian_is_second_derivative_of_row_objective():
    # g(delta) = ||delta X||^2 ; numerical second differences give 2 X X^T
    rng = np.random.default_rng(1)
    X = rng.standard_normal((4, 6))
    H = O.hessian(X)
    g = lambda d: float(np.sum((d @ X) ** 2))
    e = np.eye(4)
    h = 1e-3
    for i in range(4):
        for j in range(4):
            fd = (g(h * (e[i] + e[j])) - g(h * e[i]) - g(h * e[j]) + g(0 * e[i])) / h ** 2
            assert abs(fd - H[i, j]) < 1e-6


def test_hessian_chunks_add_up():
    rng = np.random.default_rng(2)
    X = rng.standard_normal((6, 40))
    assert np.allclose(O.hessian_from_chunks([X[:, :13], X[:, 13:29], X[:, 29:]]),
                       O.hessian(X), rtol=1e-13)


def test_damping_and_norms_conventions():
    rng = np.random.default_rng(3)
    X = rng.standard_normal((5, 20))
    H = O.hessian(X)
    Hd = O.damped(H, 0.01)
    assert np.allclose(Hd - H, 0.01 * np.trace(H) / 5 * np.eye(5))
    assert np.allclose(O.feature_norms(H), np.linalg.norm(X, axis=1))


# ---------------------------------------------------------------- single row update
def test_single_weight_update_is_obs_closed_form():
    rng = np.random.default_rng(4)
    b = 9
    X = rng.standard_normal((b, 30))
    H = O.hessian(X)
    Hinv = np.linalg.inv(H)
    w = rng.standard_normal(b)
    for q in range(b):
        delta, _ = O.row_update(Hinv, np.array([q]), w)
        want = -(w[q] / Hinv[q, q]) * Hinv[q, :]  # Eq. 3
        assert np.allclose(delta, want, rtol=1e-12, atol=1e-15)
        assert abs(O.row_loss(Hinv, H, np.array([q]), w) - 0.5 * w[q] ** 2 / Hinv[q, q]) < 1e-12


def _constrained_lstsq(w, X, q):
    """min ||(w_hat - w) X||^2 subject to w_hat[q] = 0, by a library least-squares solve
    over the free coordinates (this is the problem of Eq. 5 written out)."""
    b = w.size
    keep = np.setdiff1d(np.arange(b), q)
    target = w @ X
    sol = np.linalg.lstsq(X[keep].T, target, rcond=None)[0]
    w_hat = np.zeros(b)
    w_hat[keep] = sol
    return w_hat


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_multi_weight_update_is_constrained_least_squares(seed):
    rng = np.random.default_rng(10 + seed)
    b, a = 12, 40
    X = rng.standard_normal((b, a))
    X[3] *= 4
    w = rng.standard_normal(b)
    q = np.sort(rng.choice(b, size=rng.integers(1, 7), replace=False))
    H = O.hessian(X)
    Hinv = np.linalg.inv(H)
    delta, _ = O.row_update(Hinv, q, w)
    w_hat = w + delta
    assert np.max(np.abs(w_hat[q])) < 1e-12
    assert np.allclose(w_hat, _constrained_lstsq(w, X, q), rtol=1e-9, atol=1e-11)
    # loss of Eq. 8 equals the objective and the simplified closed form 1/2 u Rhat^-1 u^T
    S = O.row_loss(Hinv, H, q, w)
    assert abs(S - 0.5 * delta @ H @ delta) < 1e-10 * max(1, S)
    assert abs(np.sum((delta @ X) ** 2) - S) < 1e-10 * max(1, S)
    u = w[q]
    assert abs(S - 0.5 * u @ np.linalg.solve(Hinv[np.ix_(q, q)], u)) < 1e-10 * max(1, S)
    # KKT: H delta^T is supported on q only
    grad = H @ delta
    assert np.max(np.abs(np.delete(grad, q))) < 1e-9


def test_damped_update_is_least_squares_on_augmented_data():
    # 2 X' X'^T = H + lambda I for X' = [X, sqrt(lambda/2) I]: the damped update is an exact LS too
    rng = np.random.default_rng(20)
    b, a = 10, 25
    X = rng.standard_normal((b, a))
    H = O.hessian(X)
    Hd = O.damped(H, 0.05)
    lam = 0.05 * np.mean(np.diag(H))
    Xp = np.concatenate([X, math.sqrt(lam / 2) * np.eye(b)], axis=1)
    assert np.allclose(O.hessian(Xp), Hd)
    w = rng.standard_normal(b)
    q = np.array([0, 4, 7])
    delta, _ = O.row_update(np.linalg.inv(Hd), q, w)
    assert np.allclose(w + delta, _constrained_lstsq(w, Xp, q), rtol=1e-9, atol=1e-11)


# ---------------------------------------------------------------- whole sweeps
def test_unstructured_single_block_reduces_to_global_mask_plus_lstsq():
    rng = np.random.default_rng(30)
    c, b, a = 5, 10, 50
    W, X = _rand_problem(rng, c, b, a)
    p = 0.4
    Wp, M, H = O.thanos_unstructured(W, X, p, B=b, damp_rel=0.0)
    # mask: the floor(p c b) smallest |W_ij| ||X_j|| over the whole matrix
    S = np.abs(W) * np.linalg.norm(X, axis=1)[None, :]
    r = math.floor(p * c * b)
    thr = np.sort(S.ravel())[r - 1]
    assert M.sum() == r
    assert np.array_equal(M.astype(bool), S <= thr)
    for i in range(c):
        assert np.allclose(Wp[i], _constrained_lstsq(W[i], X, np.flatnonzero(M[i])),
                           rtol=1e-8, atol=1e-11)


@pytest.mark.parametrize("B", [3, 4, 8])
def test_unstructured_sweep_invariants(B):
    rng = np.random.default_rng(40 + B)
    c, b, a = 6, 16, 64
    W, X = _rand_problem(rng, c, b, a)
    p, damp = 0.55, 0.01
    steps = []
    Wp, M, H = O.thanos_unstructured(W, X, p, B, damp, collect=steps)
    # exact count, exact zeros, untouched mask convention
    assert int(M.sum()) == math.floor(p * c * b)
    assert np.all(Wp[M.astype(bool)] == 0.0)
    # each block step: the block mask is the block part of the r smallest over the residual
    xn = np.linalg.norm(X, axis=1)
    r = math.floor(p * c * b)
    for st in steps:
        j1, j2 = st["j1"], st["j2"]
        S = np.abs(st["W_before"][:, j1:]) * xn[None, j1:]
        thr = np.sort(S.ravel())[r - 1] if r > 0 else -1.0
        assert np.array_equal(st["mask"].astype(bool), (S <= thr)[:, : j2 - j1])
        r -= int(st["mask"].sum())
    assert r == 0
    # every block step is the exact constrained LS on the residual problem (damped data)
    Hd = O.damped(H, damp)
    lam = damp * np.mean(np.diag(H))
    Xp = np.concatenate([X, math.sqrt(lam / 2) * np.eye(b)], axis=1)
    for k, st in enumerate(steps):
        j1 = st["j1"]
        W_after = steps[k + 1]["W_before"] if k + 1 < len(steps) else Wp
        for i in range(c):
            q = np.flatnonzero(st["mask"][i])
            want = _constrained_lstsq(st["W_before"][i, j1:], Xp[j1:], q)
            assert np.allclose(W_after[i, j1:], want, rtol=1e-7, atol=1e-10)
            # columns left of the block are final
            assert np.array_equal(W_after[i, :j1], st["W_before"][i, :j1])
    # Pythagorean identity: block increments are H_d-orthogonal, so the total damped
    # objective is the sum of the per-row closed-form losses of all blocks
    total = O.objective_H(Wp, W, Hd)
    assert abs(total - sum(st["loss"] for st in steps)) < 1e-9 * max(1.0, total)
    assert abs(O.objective(Wp, W, Xp) - total) < 1e-9 * max(1.0, total)


def test_update_beats_plain_zeroing_with_same_mask():
    rng = np.random.default_rng(50)
    c, b, a = 8, 24, 96
    W, X = _rand_problem(rng, c, b, a, corr=1.0)
    Wp, M, H = O.thanos_unstructured(W, X, 0.5, B=b, damp_rel=0.0)
    assert O.objective(Wp, W, X) <= O.objective(O.zero_without_update(W, M), W, X) + 1e-12
    # multi-block: holds on these fixed seeds (an expectation, not a theorem)
    Wp, M, H = O.thanos_unstructured(W, X, 0.5, B=8, damp_rel=0.01)
    assert O.objective(Wp, W, X) < O.objective(O.zero_without_update(W, M), W, X)
    Wp, M, H = O.thanos_nm(W, X, 2, 4, B=8, damp_rel=0.01)
    assert O.objective(Wp, W, X) < O.objective(O.zero_without_update(W, M), W, X)


@pytest.mark.parametrize("n,m,B", [(2, 4, 8), (4, 8, 8), (1, 4, 4), (2, 4, 12)])
def test_nm_sweep_pattern_and_optimality(n, m, B):
    rng = np.random.default_rng(60 + n + m + B)
    c, b, a = 5, 24, 80
    W, X = _rand_problem(rng, c, b, a)
    steps = []
    Wp, M, H = O.thanos_nm(W, X, n, m, B, damp_rel=0.01, collect=steps)
    # every aligned group of m consecutive weights has exactly n zeros
    assert np.all(M.reshape(c, b // m, m).sum(axis=2) == n)
    assert np.all(Wp[M.astype(bool)] == 0.0)
    assert np.all(Wp[~M.astype(bool)] != 0.0)
    xn = np.linalg.norm(X, axis=1)
    for st in steps:
        j1, j2 = st["j1"], st["j2"]
        S = np.abs(st["W_before"][:, j1:j2]) * xn[None, j1:j2]
        for i in range(c):
            for g0 in range(0, j2 - j1, m):
                sel = st["mask"][i, g0:g0 + m].astype(bool)
                assert S[i, g0:g0 + m][sel].max() <= S[i, g0:g0 + m][~sel].min()
    Hd = O.damped(H, 0.01)
    total = O.objective_H(Wp, W, Hd)
    assert abs(total - sum(st["loss"] for st in steps)) < 1e-9 * max(1.0, total)


def test_tie_break_is_row_then_column():
    W = np.array([[1.0, -1.0, 2.0], [1.0, 1.0, -1.0]])
    xn = np.array([1.0, 1.0, 1.0])
    # five entries tie at metric 1; row-major order decides
    assert np.array_equal(O.psi(W, xn, 3), [[1, 1, 0], [1, 0, 0]])
    M = O.nm_block_mask(np.array([[1.0, 1.0, 1.0, 1.0]]), np.ones(4), 2, 4)
    assert np.array_equal(M, [[1, 1, 0, 0]])


def test_dead_feature_is_pruned_first():
    rng = np.random.default_rng(70)
    c, b, a = 4, 8, 30
    W, X = _rand_problem(rng, c, b, a)
    X[2] = 0.0
    Wp, M, H = O.thanos_unstructured(W, X, 0.25, 4, damp_rel=0.01)
    assert np.all(M[:, 2] == 1)


# ---------------------------------------------------------------- fast route == literal route
def test_residual_inverse_identity():
    rng = np.random.default_rng(80)
    b = 14
    A = rng.standard_normal((b, 3 * b))
    Hd = 2 * A @ A.T + 0.1 * np.eye(b)
    U = O.inverse_factor(Hd)
    assert np.allclose(np.triu(U), U)
    for j in range(b):
        assert np.allclose(np.linalg.inv(Hd[j:, j:]), U[j:, j:].T @ U[j:, j:], rtol=1e-9,
                           atol=1e-12)
    # U is the inverse of the upper factor V of the reversed-order Cholesky Hd = V V^T
    J = np.eye(b)[::-1]
    V = J @ np.linalg.cholesky(J @ Hd @ J) @ J
    assert np.allclose(V @ V.T, Hd)
    assert np.allclose(U, np.linalg.inv(V), rtol=1e-9, atol=1e-12)


@pytest.mark.parametrize("mode", ["unstructured", "nm"])
def test_fast_sweep_equals_literal_sweep(mode):
    rng = np.random.default_rng(90)
    c, b, a = 12, 40, 160
    W, X = _rand_problem(rng, c, b, a)
    if mode == "unstructured":
        Wl, Ml, _ = O.thanos_unstructured(W, X, 0.5, 8, 0.01)
        Wf, Mf, _ = O.thanos_unstructured_fast(W, X, 0.5, 8, 0.01)
    else:
        Wl, Ml, _ = O.thanos_nm(W, X, 2, 4, 8, 0.01)
        Wf, Mf, _ = O.thanos_nm_fast(W, X, 2, 4, 8, 0.01)
    assert np.array_equal(Ml, Mf)
    assert np.max(np.abs(Wl - Wf)) <= 1e-10 * np.max(np.abs(Wl))
    Hd = O.damped(O.hessian(X), 0.01)
    rows = [0, 5, 11]
    Wr = O.replay_rows(W[rows], Ml[rows], Hd, 8)
    assert np.max(np.abs(Wr - Wl[rows])) <= 1e-10 * np.max(np.abs(Wl))


def test_ragged_last_block_and_p_zero():
    rng = np.random.default_rng(95)
    c, b, a = 4, 11, 50
    W, X = _rand_problem(rng, c, b, a)
    Wp, M, _ = O.thanos_unstructured(W, X, 0.3, 4, 0.01)  # blocks 4,4,3
    assert int(M.sum()) == math.floor(0.3 * c * b)
    Wp0, M0, _ = O.thanos_unstructured(W, X, 0.0, 4, 0.01)
    assert M0.sum() == 0 and np.array_equal(Wp0, W)


# ------------------------------------------------------------------------------ outlier rows
def test_row_losses_match_their_definition_and_the_hessian_form():
    rng = np.random.default_rng(5)
    W = rng.standard_normal((7, 12))
    X = rng.standard_normal((12, 40))
    h_def = np.array([np.linalg.norm(W[i] @ X) ** 2 for i in range(7)])   # ||W_i X||_2^2
    assert np.allclose(O.row_losses(W, X=X), h_def, rtol=1e-12)
    assert np.allclose(O.row_losses(W, H=O.hessian(X)), h_def, rtol=1e-12)
    # removing row i entirely costs exactly h_i in the objective of Eq. 1
    for i in (0, 3):
        Wh = W.copy()
        Wh[i] = 0.0
        assert abs(O.objective(Wh, W, X) - h_def[i]) <= 1e-9 * h_def[i]


def test_outlier_rows_are_the_largest_losses_and_stay_untouched():
    rng = np.random.default_rng(6)
    c, b, B = 10, 16, 8
    W = rng.standard_normal((c, b))
    X = rng.standard_normal((b, 64))
    W[2] *= 30.0
    W[7] *= 20.0                                   # two rows with by far the largest h_i
    alpha = 0.15                                   # ceil(1.5) = 2 outlier rows
    Wp, M, H = O.thanos_nm(W, X, 2, 4, B, 0.01, alpha=alpha)
    h = O.row_losses(W, X=X)
    sigma, n_out = O.outlier_row_order(h, alpha)
    assert n_out == 2 and set(sigma[-2:]) == {2, 7}
    assert np.array_equal(Wp[[2, 7]], W[[2, 7]]) and M[[2, 7]].sum() == 0
    # the other rows are pruned exactly as without outliers: rows are independent in n:m mode
    W0, M0, _ = O.thanos_nm(W, X, 2, 4, B, 0.01)
    keep = np.array([i for i in range(c) if i not in (2, 7)])
    assert np.array_equal(M[keep], M0[keep]) and np.allclose(Wp[keep], W0[keep], rtol=0, atol=1e-12)
    assert int(M.sum()) == (c - 2) * b // 2
    # alpha = 0 is the plain algorithm; ties in h keep row order (stable)
    Wz, Mz, _ = O.thanos_nm(W, X, 2, 4, B, 0.01, alpha=0.0)
    assert np.array_equal(Mz, M0) and np.array_equal(Wz, W0)
    s2, n2 = O.outlier_row_order(np.array([1.0, 3.0, 3.0, 0.5]), 0.25)
    assert n2 == 1 and list(s2) == [3, 0, 1, 2]    # of the tied rows 1 and 2, row 2 is the outlier


# ------------------------------------------------------------------------------ structured
def test_column_losses_match_the_frobenius_definition():
    rng = np.random.default_rng(8)
    W = rng.standard_normal((5, 7))
    X = rng.standard_normal((7, 30))
    xn = O.feature_norms(O.hessian(X))
    v = O.column_losses(W, xn)
    for j in range(7):
        outer = np.outer(W[:, j], X[j])             # W_{:, j} (x) X_j
        assert abs(v[j] - np.linalg.norm(outer, "fro") ** 2) <= 1e-10 * v[j]
    assert O.structured_column_count(0.3, 10, 0.0) == 3
    assert O.structured_column_count(0.3, 10, 0.25) == 4     # ceil(3 / 0.75)
    assert O.structured_column_count(0.25, 10, 0.0) == 3     # ceil(2.5): rounded up
    assert O.structured_column_count(0.5, 7, 0.1) == 4       # ceil(3.5 / 0.9) = ceil(3.89)


def test_structured_is_the_constrained_least_squares_refit():
    """Pruned rows: zeros in the s removed columns, and the kept columns minimise
    ||(w_hat - w) X'||^2 (X' = X with the damping appended) -- a plain lstsq; outlier rows are
    returned unchanged; the removed columns are the s smallest v_j."""
    rng = np.random.default_rng(9)
    c, b, a = 9, 14, 60
    W = rng.standard_normal((c, b))
    X = rng.standard_normal((b, a)) * rng.uniform(0.5, 2.0, size=(b, 1))
    W[4] *= 25.0
    for alpha, p in ((0.0, 0.3), (0.1, 0.25)):
        Wp, removed, outl, H = O.thanos_structured(W, X, p, alpha, damp_rel=0.02)
        s = O.structured_column_count(p, b, alpha)
        assert removed.sum() == s
        n_out = int(math.ceil(alpha * c - 1e-12)) if alpha > 0 else 0
        assert outl.sum() == n_out and (n_out == 0 or outl[4])
        assert np.array_equal(Wp[outl], W[outl])
        rows = ~outl
        assert np.all(Wp[np.ix_(rows, removed)] == 0.0)
        v = O.column_losses(W[rows], O.feature_norms(H))
        assert v[removed].max() <= v[~removed].min()
        lam = 0.02 * np.mean(np.diag(H))
        Xd = np.concatenate([X, np.sqrt(lam / 2.0) * np.eye(b)], axis=1)   # 2 Xd Xd^T = H + lam I
        keep = ~removed
        for i in np.nonzero(rows)[0]:
            sol, *_ = np.linalg.lstsq(Xd[keep].T, (W[i] @ Xd), rcond=None)
            assert np.allclose(Wp[i, keep], sol, rtol=1e-8, atol=1e-10)


def test_structured_single_column_is_the_obs_closed_form():
    rng = np.random.default_rng(10)
    c, b = 3, 6
    W = rng.standard_normal((c, b))
    X = rng.standard_normal((b, 40))
    Wp, removed, outl, H = O.thanos_structured(W, X, 1.0 / b, 0.0, damp_rel=0.0)
    q = int(np.nonzero(removed)[0][0])
    Hinv = np.linalg.inv(H)
    for i in range(c):
        want = W[i] - (W[i, q] / Hinv[q, q]) * Hinv[q]      # Eq. 3
        want[q] = 0.0
        assert np.allclose(Wp[i], want, rtol=1e-9, atol=1e-12)


def test_structured_update_rows_agrees_with_algorithm_2():
    rng = np.random.default_rng(11)
    W = rng.standard_normal((6, 12))
    X = rng.standard_normal((12, 50))
    Wp, removed, outl, H = O.thanos_structured(W, X, 0.25, 0.0, damp_rel=0.01)
    rows = O.structured_update_rows(W[[1, 4]], removed, O.damped(H, 0.01))
    assert np.allclose(rows, Wp[[1, 4]], rtol=1e-10, atol=1e-12)
