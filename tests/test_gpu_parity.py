"""GPU parity tests: the CUDA library (through its C ABI) against the float64 oracle on the same
seeded inputs."""

import math

import numpy as np
import pytest
import torch

import workloads as WL
from oracle import thanos_oracle as O
from tests import parity_utils as PU

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def T():
    import paper_2504_05346_b200 as T_
    from paper_2504_05346_b200 import build as B_

    B_.build()
    T_.load_library()
    return T_


DEV = "cuda"


def _np64(t):
    return t.detach().cpu().double().numpy()


def _acts(a, b, dtype, dist="student_t4", frac=0.01, count=0, scale=20.0, seed=7, mix=0.0):
    return WL.make_activations(a, b, dtype, dist, frac, count, scale, seed, 0, mix=mix)


def _gpu_hessian(T, Xt, chunks=1):
    b = Xt.shape[1]
    H = torch.zeros((b, b), dtype=torch.float32, device=DEV)
    Xd = Xt.to(DEV)
    edges = np.linspace(0, Xt.shape[0], chunks + 1).astype(int)
    for k in range(chunks):
        T.hessian_accumulate(H, Xd[edges[k]:edges[k + 1]])
    return H


# ------------------------------------------------------------------------------ Hessian
@pytest.mark.parametrize("dtype,b,n_tok,chunks", [
    ("f32", 256, 2048, 2), ("bf16", 264, 1000, 3), ("f32", 8, 5, 1), ("bf16", 1024, 4113, 1),
    ("f32", 136, 777, 4), ("bf16", 4096, 1024, 1)])
def test_hessian_parity(T, dtype, b, n_tok, chunks):
    Xt = _acts(n_tok, b, dtype, seed=11 + b)
    H = _gpu_hessian(T, Xt, chunks)
    Ho = O.hessian(_np64(Xt).T)
    Hg = _np64(H)
    assert PU.rel_fro(Hg, Ho) <= PU.TOL_H
    assert np.max(np.abs(Hg - Hg.T)) <= 1e-5 * np.max(np.abs(Hg))
    # per-entry check on the diagonal (the metric norms come from it)
    assert np.max(np.abs(np.diag(Hg) - np.diag(Ho)) / np.diag(Ho)) <= 1e-5


def test_hessian_strided_input_and_empty_chunk(T):
    Xfull = _acts(512, 320, "f32", seed=5)
    Xd = Xfull.to(DEV)
    view = Xd[:, :192]  # leading dimension 320, 192 columns
    H = torch.zeros((192, 192), dtype=torch.float32, device=DEV)
    T.hessian_accumulate(H, view)
    T.hessian_accumulate(H, view[:0])
    Ho = O.hessian(_np64(Xfull[:, :192]).T)
    assert PU.rel_fro(_np64(H), Ho) <= PU.TOL_H


@pytest.mark.parametrize("b,n_tok,dtype", [(4096, 32768, "bf16"), (11008, 12345, "bf16"),
                                           (768, 70001 // 8 * 8, "f32"), (3072, 20000, "f32")])
def test_hessian_bench_shape_sampled(T, b, n_tok, dtype):
    """The benchmark's layer widths with long chunks (bf16: CTA-pair kernel, several token slices,
    a ragged token tail; fp32: the widths of the OPT-125M-shaped set, more tokens than one pass of
    the split into planes takes, stages that hold all three planes): sampled entries against a
    float64 dot product."""
    Xd = WL.make_activations(n_tok, b, dtype, "student_t4", 0.005, 0, 50.0, 2, 0, device=DEV)
    H = torch.zeros((b, b), dtype=torch.float32, device=DEV)
    T.hessian_accumulate(H, Xd)
    torch.cuda.synchronize()
    rng = np.random.default_rng(0)
    ii = rng.integers(0, b, 48)
    jj = rng.integers(0, b, 48)
    ii[:8] = jj[:8]  # some diagonal entries
    outl = WL.outlier_channels(b, 0.005, 0, 2, 0).numpy()
    ii[8:12] = outl[:4]
    cols = np.unique(np.concatenate([ii, jj]))
    Xc = _np64(Xd[:, torch.as_tensor(cols, device=DEV)])
    pos = {c_: k for k, c_ in enumerate(cols)}
    Hs = _np64(H[torch.as_tensor(ii, device=DEV), torch.as_tensor(jj, device=DEV)])
    want = np.array([2.0 * np.dot(Xc[:, pos[i]], Xc[:, pos[j]]) for i, j in zip(ii, jj)])
    scale = np.sqrt(np.array([2.0 * np.dot(Xc[:, pos[i]], Xc[:, pos[i]]) *
                              2.0 * np.dot(Xc[:, pos[j]], Xc[:, pos[j]]) for i, j in zip(ii, jj)]))
    assert np.max(np.abs(Hs - want) / scale) <= 1e-5
    Hh = H.cpu()
    assert torch.equal(torch.isfinite(Hh).all(), torch.tensor(True))
    assert float((Hh - Hh.T).abs().max()) <= 1e-5 * float(Hh.abs().max())


# ------------------------------------------------------------------------------ factor
@pytest.mark.parametrize("b,mix", [(64, 0.0), (200, 0.5), (256, 0.0), (520, 1.0), (1024, 0.3)])
def test_prepare_inverse_parity(T, b, mix):
    Xt = _acts(4 * b, b, "f32", seed=3 + b, mix=mix)
    Ho = O.hessian(_np64(Xt).T)
    H = torch.tensor(Ho, dtype=torch.float32, device=DEV)
    H64 = _np64(H)
    U, xn = T.prepare_inverse(H, 0.01)
    Ug = _np64(U)
    assert np.all(np.tril(Ug, -1) == 0.0)
    Hd = O.damped(H64, 0.01)
    Uo = O.inverse_factor(Hd)
    assert PU.rel_fro(Ug, Uo) <= 2e-4
    Hinv = np.linalg.inv(Hd)
    assert PU.rel_fro(Ug.T @ Ug, Hinv) <= 2e-4
    for j in (0, b // 3, b - 5):
        assert PU.rel_fro(Ug[j:, j:].T @ Ug[j:, j:], np.linalg.inv(Hd[j:, j:])) <= 2e-4
    assert np.allclose(_np64(xn), O.feature_norms(H64), rtol=1e-6)


def test_prepare_inverse_reports_singular_matrix(T):
    b = 64
    Xt = _acts(16, b, "f32", seed=1)  # rank 16 < b
    H = torch.tensor(O.hessian(_np64(Xt).T), dtype=torch.float32, device=DEV)
    with pytest.raises(T.ThanosError) as e:
        T.prepare_inverse(H, 0.0)
    assert e.value.code == 6  # THANOS_ERR_NOT_SPD
    U, xn = T.prepare_inverse(H, 0.01)  # damping makes it positive definite
    assert torch.isfinite(U).all()


def test_prepare_inverse_4096_sampled(T):
    """Bench-size factor: columns of inv(H_d[j:, j:]) from U against float64 solves."""
    b = 4096
    Xd = WL.make_activations(16384, b, "bf16", "student_t4", 0.005, 0, 50.0, 2, 0, device=DEV)
    H = torch.zeros((b, b), dtype=torch.float32, device=DEV)
    T.hessian_accumulate(H, Xd)
    U, xn = T.prepare_inverse(H, 0.01)
    Hd = O.damped(_np64(H), 0.01)
    Ug = _np64(U)
    for j0, col in ((0, 17), (0, 4000), (2048, 5), (3968, 100)):
        e = np.zeros(b - j0)
        e[col] = 1.0
        want = np.linalg.solve(Hd[j0:, j0:], e)
        got = Ug[j0:, j0:].T @ Ug[j0:, j0 + col]
        assert np.linalg.norm(got - want) <= 2e-4 * np.linalg.norm(want)


# ------------------------------------------------------------------------------ whole sweep
def _oracle_sweep(W64, H64, mode, p, n, m, B, damp, literal):
    steps = [] if literal else None
    if mode == "unstructured":
        fn = O.thanos_unstructured if literal else O.thanos_unstructured_fast
        args = (W64, None, p, B, damp)
    else:
        fn = O.thanos_nm if literal else O.thanos_nm_fast
        args = (W64, None, n, m, B, damp)
    if literal:
        Wo, Mo, _ = fn(*args, H=H64, collect=steps)
    else:
        Wo, Mo, _ = fn(*args, H=H64)
    return Wo, Mo, steps


def _check_sweep(T, W, H, mode, p, n, m, B, damp, tolW, literal=True, tolD=2e-3):
    """Runs prepare_inverse + prune_layer on (W, H) and the oracle on the same H; returns
    diagnostics after asserting the parity protocol."""
    c, b = W.shape
    Wd = W.to(DEV)
    U, xn = T.prepare_inverse(H, damp)
    if mode == "unstructured":
        Wp, M, st = T.prune_layer(Wd, U, xn, T.UNSTRUCTURED, p=p, B=B)
    else:
        Wp, M, st = T.prune_layer(Wd, U, xn, T.NM, n=n, m=m, B=B)
    torch.cuda.synchronize()
    H64, W64 = _np64(H), _np64(W)
    Wo, Mo, steps = _oracle_sweep(W64, H64, mode, p, n, m, B, damp, literal)
    Mg, Wg = M.cpu().numpy(), _np64(Wp)
    # structural facts that hold whatever the ties do
    assert np.all(Wg[Mg.astype(bool)] == 0.0)
    if mode == "unstructured":
        assert int(Mg.sum()) == PU.expected_removed(p, c, b) == st.n_pruned
        assert st.r_left == 0
    else:
        assert np.all(Mg.reshape(c, b // m, m).sum(axis=2) == n)
        assert st.n_pruned == c * b // m * n
    assert st.n_blocks == math.ceil(b / B)
    # mask: exact, except near-ties.  Unstructured: the first block that differs is classified
    # (one flip moves every later threshold).  n:m: rows are independent, so every row is
    # classified in the first block where it differs.
    near = bad = 0
    diff = Mg != Mo
    if diff.any():
        assert steps is not None, "mask differs and no per-block oracle state was kept"
        xn64 = O.feature_norms(H64)
        r = PU.expected_removed(p, c, b) if mode == "unstructured" else 0
        clean = np.ones(c, dtype=bool)
        for stp in steps:
            j1, j2 = stp["j1"], stp["j2"]
            d = diff[:, j1:j2]
            if mode == "unstructured":
                if d.any():
                    tau, S = PU.block_threshold(stp["W_before"], xn64, j1, stp["mask"], r)
                    near, bad = PU.classify_unstructured_block(Mg[:, j1:j2], stp["mask"],
                                                               S[:, : j2 - j1], tau)
                    break
                r -= int(stp["mask"].sum())
            else:
                rows = clean & d.any(axis=1)
                if rows.any():
                    S = np.abs(stp["W_before"][rows][:, j1:j2]) * xn64[None, j1:j2]
                    nk, bk = PU.classify_nm_block(Mg[rows][:, j1:j2], stp["mask"][rows], S, n, m)
                    near += nk
                    bad += bk
                clean &= ~d.any(axis=1)
        assert bad == 0, "mask mismatch that is not a near-tie: %d (near-ties %d)" % (bad, near)
    # weights: rows whose masks agree follow the same updates
    same = ~diff.any(axis=1)
    assert same.sum() >= 0.9 * c
    if W.dtype == torch.bfloat16:
        Wo_cmp = _np64(torch.tensor(Wo).to(torch.bfloat16))
    else:
        Wo_cmp = Wo
    relW = PU.rel_fro(Wg[same], Wo_cmp[same])
    assert relW <= tolW, relW
    out = {"relW": relW, "near": near, "mismatch": int(diff.sum()), "stats": st}
    if W.dtype == torch.float32:
        Dg = Wg - (1 - Mg) * W64
        Do = Wo - (1 - Mo) * W64
        relD = PU.rel_fro(Dg[same], Do[same])
        assert relD <= tolD, relD
        Hd = O.damped(H64, damp)
        eg, eo = O.objective_H(Wg[same], W64[same], Hd), O.objective_H(Wo[same], W64[same], Hd)
        assert abs(eg / eo - 1.0) <= 1e-3
        out["relD"] = relD
    return out


def test_config_tiny_exact(T):
    """The smallest benchmark configuration, end to end (Hessian included)."""
    cfg = WL.CONFIGS["tiny"]
    L = cfg.layers[0]
    W = WL.config_weight(cfg, 0)
    Xt = WL.config_activations(cfg, 0, L.b)
    H = _gpu_hessian(T, Xt, chunks=2)
    Ho = O.hessian(_np64(Xt).T)
    assert PU.rel_fro(_np64(H), Ho) <= PU.TOL_H
    r = _check_sweep(T, W, H, "unstructured", cfg.p, 0, 0, cfg.B, cfg.damp_rel, PU.TOL_W_F32)
    # and against the oracle run on its own float64 Hessian
    Wo, Mo, _ = O.thanos_unstructured(_np64(W), _np64(Xt).T, cfg.p, cfg.B, cfg.damp_rel)
    U, xn = T.prepare_inverse(H, cfg.damp_rel)
    Wp, M, st = T.prune_layer(W.to(DEV), U, xn, T.UNSTRUCTURED, p=cfg.p, B=cfg.B)
    assert int((M.cpu().numpy() != Mo).sum()) <= 8
    same = ~(M.cpu().numpy() != Mo).any(axis=1)
    assert PU.rel_fro(_np64(Wp)[same], Wo[same]) <= PU.TOL_W_F32


SWEEP_CASES = [
    # name, c, b, a, dtype, dist, mode, p, n, m, B, mix
    ("opt_like_2of4", 192, 384, 4096, "f32", "student_t4", "nm", 0.0, 2, 4, 128, 0.0),
    ("opt_like_2of4_mix", 384, 256, 4096, "f32", "student_t4", "nm", 0.0, 2, 4, 128, 1.0),
    ("llama2_like_unstr", 320, 512, 8192, "bf16", "student_t4", "unstructured", 0.5, 0, 0, 128, 0.0),
    ("llama2_like_unstr_mix", 160, 384, 4096, "bf16", "student_t4", "unstructured", 0.5, 0, 0, 128, 0.7),
    ("llama3_like_4of8", 256, 512, 8192, "bf16", "student_t4", "nm", 0.0, 4, 8, 256, 0.0),
    ("l70b_like_2of4", 128, 1024, 4096, "bf16", "student_t4", "nm", 0.0, 2, 4, 128, 0.0),
    ("l70b_like_unstr60", 128, 1024, 4096, "bf16", "student_t4", "unstructured", 0.6, 0, 0, 128, 0.0),
    ("f32_unstr_mix", 200, 320, 2048, "f32", "normal", "unstructured", 0.5, 0, 0, 64, 1.0),
    ("ragged_unstr", 77, 328, 2048, "f32", "normal", "unstructured", 0.37, 0, 0, 64, 0.5),
    ("ragged_nm", 77, 328, 2048, "f32", "normal", "nm", 0.0, 1, 4, 64, 0.5),
    ("wide_block_unstr", 64, 512, 4096, "f32", "student_t4", "unstructured", 0.5, 0, 0, 256, 0.3),
    ("b512_2of4", 48, 1024, 4096, "f32", "student_t4", "nm", 0.0, 2, 4, 512, 0.3),
    ("small_block", 40, 64, 512, "f32", "normal", "unstructured", 0.5, 0, 0, 8, 0.5),
    ("b512_unstr", 300, 1024, 4096, "f32", "student_t4", "unstructured", 0.5, 0, 0, 512, 0.3),
    ("b512_unstr70", 160, 1024, 4096, "bf16", "student_t4", "unstructured", 0.7, 0, 0, 512, 0.3),
    ("b400_unstr", 90, 1200, 4096, "f32", "normal", "unstructured", 0.45, 0, 0, 400, 0.5),
    ("b512_4of8", 200, 512, 4096, "bf16", "student_t4", "nm", 0.0, 4, 8, 512, 0.0),
    ("grouped_2of4", 96, 2304, 4096, "f32", "student_t4", "nm", 0.0, 2, 4, 128, 0.3),
    ("grouped_4of8_b256", 72, 2176, 4096, "bf16", "normal", "nm", 0.0, 4, 8, 256, 0.5),
]


@pytest.mark.parametrize("case", SWEEP_CASES, ids=[c[0] for c in SWEEP_CASES])
def test_sweep_parity(T, case):
    name, c, b, a, dtype, dist, mode, p, n, m, B, mix = case
    W = WL.make_weight(c, b, dtype, seed=21, layer_index=len(name))
    Xt = WL.make_activations(a, b, dtype, dist, 0.01, 0, 20.0, 13, len(name), mix=mix)
    H = _gpu_hessian(T, Xt, chunks=2)
    assert PU.rel_fro(_np64(H), O.hessian(_np64(Xt).T)) <= PU.TOL_H
    tol = PU.TOL_W_BF16 if dtype == "bf16" else PU.TOL_W_F32
    _check_sweep(T, W, H, mode, p, n, m, B, 0.01, tol)


# ------------------------------------------------------------------------------ block steps
@pytest.mark.parametrize("mode", ["unstructured", "nm"])
def test_block_step_teacher_forced(T, mode):
    """Every block step from the ORACLE's state: mask of the block, then the updated weights."""
    c, b, B = 96, 256, 64
    W = WL.make_weight(c, b, "f32", seed=31)
    Xt = WL.make_activations(2048, b, "f32", "student_t4", 0.02, 0, 10.0, 17, 0, mix=0.6)
    H = _gpu_hessian(T, Xt)
    H64 = _np64(H)
    p, n, m = 0.5, 2, 4
    steps = []
    if mode == "unstructured":
        Wo, Mo, _ = O.thanos_unstructured(_np64(W), None, p, B, 0.01, H=H64, collect=steps)
    else:
        Wo, Mo, _ = O.thanos_nm(_np64(W), None, n, m, B, 0.01, H=H64, collect=steps)
    U, xn = T.prepare_inverse(H, 0.01)
    xn64 = O.feature_norms(H64)
    r = PU.expected_removed(p, c, b)
    for k, stp in enumerate(steps):
        j1, j2 = stp["j1"], stp["j2"]
        Wc = torch.tensor(stp["W_before"], dtype=torch.float32, device=DEV)
        mask = torch.zeros((c, b), dtype=torch.uint8, device=DEV)
        stats = torch.zeros(64, dtype=torch.uint8, device=DEV)
        rt = torch.tensor([r], dtype=torch.int64, device=DEV)
        T.prune_block(Wc, mask, U, xn, T.UNSTRUCTURED if mode == "unstructured" else T.NM,
                      n, m, B, j1, rt if mode == "unstructured" else None, stats)
        torch.cuda.synchronize()
        Mg = mask.cpu().numpy()[:, j1:j2]
        if mode == "unstructured":
            tau, S = PU.block_threshold(stp["W_before"], xn64, j1, stp["mask"], r)
            near, bad = PU.classify_unstructured_block(Mg, stp["mask"], S[:, : j2 - j1], tau)
            assert int(rt.item()) == r - int(Mg.sum())
        else:
            S = np.abs(stp["W_before"][:, j1:j2]) * xn64[None, j1:j2]
            near, bad = PU.classify_nm_block(Mg, stp["mask"], S, n, m)
        assert bad == 0 and near <= 2
        W_after = steps[k + 1]["W_before"] if k + 1 < len(steps) else Wo
        same = ~(Mg != stp["mask"]).any(axis=1)
        Wg = _np64(Wc)
        assert np.array_equal(Wg[:, :j1], stp["W_before"].astype(np.float32)[:, :j1])
        assert PU.rel_fro(Wg[same][:, j1:], W_after[same][:, j1:]) <= 2e-5
        D_or = W_after[same][:, j1:] - stp["W_before"][same][:, j1:]
        D_g = Wg[same][:, j1:] - stp["W_before"].astype(np.float32).astype(np.float64)[same][:, j1:]
        assert PU.rel_fro(D_g, D_or) <= 1e-3
        r -= int(stp["mask"].sum())


# ------------------------------------------------------------------------------ edge cases
def _equal_norm_hessian(b, a=4096.0, seed=0):
    """A synthetic SPD Hessian with a constant diagonal, so the metric reduces to |W| times a
    constant and exact ties in W are exact ties in the metric."""
    rng = np.random.default_rng(seed)
    A = rng.standard_normal((b, 8))
    C = A @ A.T
    d = np.sqrt(np.diag(C))
    C = C / d[:, None] / d[None, :]
    H = 2.0 * a * (0.7 * np.eye(b) + 0.3 * C)
    return torch.tensor(H, dtype=torch.float32)


def test_exact_ties_follow_row_then_column_order(T):
    c, b, B = 64, 128, 32
    H = _equal_norm_hessian(b)
    Hd = H.to(DEV)
    d = torch.diag(H)
    assert float(d.max() - d.min()) == 0.0
    g = torch.Generator().manual_seed(3)
    W = (torch.randint(-4, 5, (c, b), generator=g).float() * 0.01)
    U, xn = T.prepare_inverse(Hd, 0.01)
    Wp, M, st = T.prune_layer(W.to(DEV), U, xn, T.UNSTRUCTURED, p=0.5, B=B)
    steps = []
    Wo, Mo, _ = O.thanos_unstructured(_np64(W), None, 0.5, B, 0.01, H=_np64(H), collect=steps)
    Mg = M.cpu().numpy()
    # the first block is decided on the raw grid values: it must match bit for bit
    assert np.array_equal(Mg[:, :B], Mo[:, :B])
    assert int(Mg.sum()) == PU.expected_removed(0.5, c, b)
    assert st.n_tied > 0
    # n:m on the same grid: ties inside groups go to the lower column
    Wp2, M2, _ = T.prune_layer(W.to(DEV), U, xn, T.NM, n=2, m=4, B=B)
    Wo2, Mo2, _ = O.thanos_nm(_np64(W), None, 2, 4, B, 0.01, H=_np64(H))
    assert np.array_equal(M2.cpu().numpy()[:, :B], Mo2[:, :B])


def test_rows_with_no_and_all_removals_and_dead_feature(T):
    c, b, B = 32, 128, 32
    W = WL.make_weight(c, b, "f32", seed=41)
    W[0] *= 1e-4   # every entry of row 0 goes: s = B in every block
    W[1] *= 1e3    # nothing of row 1 goes: s = 0
    Xt = WL.make_activations(1024, b, "f32", "normal", 0.0, 2, 20.0, 19, 0, mix=0.4)
    Xt[:, 5] = 0.0  # dead input feature: metric 0, always removed
    H = _gpu_hessian(T, Xt)
    r = _check_sweep(T, W, H, "unstructured", 0.5, 0, 0, B, 0.01, PU.TOL_W_F32)
    U, xn = T.prepare_inverse(H, 0.01)
    Wp, M, st = T.prune_layer(W.to(DEV), U, xn, T.UNSTRUCTURED, p=0.5, B=B)
    Mg = M.cpu().numpy()
    assert Mg[0].all() and Mg[:, 5].all()
    assert Mg[1].sum() <= 4 and not Mg[1, 32:64].any()  # only the dead feature and stragglers
    assert st.max_s == B
    # a row receives no update in a block where nothing of it is removed
    assert np.array_equal(_np64(Wp)[1, 32:64] != 0, np.ones(32, bool))


def test_p_zero_is_identity(T):
    c, b = 16, 64
    W = WL.make_weight(c, b, "bf16", seed=43)
    H = _equal_norm_hessian(b).to(DEV)
    U, xn = T.prepare_inverse(H, 0.01)
    Wp, M, st = T.prune_layer(W.to(DEV), U, xn, T.UNSTRUCTURED, p=0.0, B=32)
    assert int(M.sum()) == 0 and torch.equal(Wp.cpu(), W) and st.n_pruned == 0


def test_in_place_output(T):
    c, b = 24, 96
    W = WL.make_weight(c, b, "f32", seed=47)
    H = _equal_norm_hessian(b, seed=2).to(DEV)
    U, xn = T.prepare_inverse(H, 0.01)
    Wd = W.to(DEV)
    Wp, M, _ = T.prune_layer(Wd, U, xn, T.NM, n=2, m=4, B=32)
    Wd2 = W.to(DEV)
    Wp2, M2, _ = T.prune_layer(Wd2, U, xn, T.NM, n=2, m=4, B=32, out=Wd2)
    assert Wp2.data_ptr() == Wd2.data_ptr()
    assert torch.equal(Wp, Wp2) and torch.equal(M, M2)


def test_sweep_is_deterministic(T):
    c, b = 96, 256
    W = WL.make_weight(c, b, "bf16", seed=53)
    Xt = _acts(2048, b, "bf16", seed=9, mix=0.5)
    H = _gpu_hessian(T, Xt)
    U, xn = T.prepare_inverse(H, 0.01)
    U2, xn2 = T.prepare_inverse(H, 0.01)
    assert torch.equal(U, U2) and torch.equal(xn, xn2)
    a = T.prune_layer(W.to(DEV), U, xn, T.UNSTRUCTURED, p=0.5, B=64)
    b_ = T.prune_layer(W.to(DEV), U, xn, T.UNSTRUCTURED, p=0.5, B=64)
    assert torch.equal(a[0], b_[0]) and torch.equal(a[1], b_[1])


@pytest.mark.parametrize("dtype,b,a", [("bf16", 1024, 20000), ("f32", 512, 9000), ("bf16", 2048, 33000)])
def test_ordered_hessian_makes_the_whole_path_reproducible(T, dtype, b, a):
    """thanos_hessian_accumulate_ordered at widths where the unordered call splits its tokens into
    concurrent slices: two runs give the same H bit for bit (and with it the same factor, masks and
    weights); the ordered H is the unordered one up to rounding."""
    c = 128
    W = WL.make_weight(c, b, dtype, seed=57)
    Xd = _acts(a, b, dtype, seed=10 + b, mix=0.3).to(DEV)
    runs = []
    for _ in range(2):
        H = torch.zeros((b, b), dtype=torch.float32, device=DEV)
        T.hessian_accumulate(H, Xd[:a // 2], ordered=True)
        T.hessian_accumulate(H, Xd[a // 2:], ordered=True)
        U, xn = T.prepare_inverse(H, 0.01)
        Wp, M, st = T.prune_layer(W.to(DEV), U, xn, T.UNSTRUCTURED, p=0.5, B=128)
        runs.append((H, U, xn, Wp, M))
    for x, y in zip(*runs):
        assert torch.equal(x, y)
    Hu = torch.zeros((b, b), dtype=torch.float32, device=DEV)
    T.hessian_accumulate(Hu, Xd)
    assert PU.rel_fro(_np64(runs[0][0]), _np64(Hu)) <= 1e-6
    assert PU.rel_fro(_np64(Hu), O.hessian(_np64(Xd).T)) <= PU.TOL_H
    assert PU.rel_fro(_np64(runs[0][0]), O.hessian(_np64(Xd).T)) <= PU.TOL_H


def test_argument_errors_are_reported(T):
    b = 64
    H = _equal_norm_hessian(b).to(DEV)
    U, xn = T.prepare_inverse(H, 0.01)
    W = WL.make_weight(8, b, "f32", seed=1).to(DEV)
    with pytest.raises(T.ThanosError) as e:
        T.prune_layer(W, U, xn, T.NM, n=2, m=4, B=30)  # B not a multiple of 8
    assert e.value.code == 2
    with pytest.raises(T.ThanosError) as e:
        T.prune_layer(W, U, xn, T.NM, n=4, m=4, B=32)  # n must be < m
    assert e.value.code == 1
    with pytest.raises(T.ThanosError) as e:
        T.prune_layer(W, U, xn, T.UNSTRUCTURED, p=1.0, B=32)
    assert e.value.code == 1
    with pytest.raises(T.ThanosError) as e:
        T.prune_layer(W, U, xn, T.UNSTRUCTURED, p=0.5, B=32,
                      workspace=torch.empty(256, dtype=torch.uint8, device=DEV))
    assert e.value.code == 5
    with pytest.raises(T.ThanosError) as e:
        T.hessian_accumulate(torch.zeros((60, 60), device=DEV), torch.zeros((4, 60), device=DEV))
    assert e.value.code == 2  # b % 8 != 0
    # the context is still usable
    Wp, M, st = T.prune_layer(W, U, xn, T.NM, n=2, m=4, B=32)
    assert st.status == 0


# ------------------------------------------------------------------------------ outlier rows
@pytest.mark.parametrize("c,b,dtype,n,m,B,alpha", [
    (96, 256, "f32", 2, 4, 64, 0.1), (160, 384, "bf16", 2, 4, 128, 0.05),
    (64, 256, "f32", 4, 8, 64, 0.3), (50, 128, "f32", 2, 4, 32, 0.0)])
def test_outlier_rows_parity(T, c, b, dtype, n, m, B, alpha):
    """Algorithm 4 with alpha: outlier flags, untouched outlier rows, and the other rows against
    the oracle (rows are independent in n:m mode)."""
    W = WL.make_weight(c, b, dtype, seed=81, layer_index=c)
    g = torch.Generator().manual_seed(c + b)
    scale = torch.exp(0.7 * torch.randn((c, 1), generator=g))   # spread the row losses
    W = (W.float() * scale).to(W.dtype)
    Xt = WL.make_activations(2048, b, dtype, "student_t4", 0.02, 0, 10.0, 29, 0, mix=0.5)
    H = _gpu_hessian(T, Xt)
    H64, W64 = _np64(H), _np64(W)
    U, xn = T.prepare_inverse(H, 0.01)
    Wp, M, flags, st = T.prune_layer_outliers(W.to(DEV), U, xn, H, n, m, alpha, B=B)
    torch.cuda.synchronize()
    # outlier rows: the ceil(alpha c) largest h_i (differences only between near-equal losses)
    h = O.row_losses(W64, H=H64)
    sigma, n_out = O.outlier_row_order(h, alpha)
    fo = np.zeros(c, dtype=np.uint8)
    fo[sigma[c - n_out:]] = 1
    fg = flags.cpu().numpy()
    assert int(fg.sum()) == n_out
    if n_out:
        hb = h[sigma[c - n_out]]                     # smallest outlier loss
        for i in np.nonzero(fg != fo)[0]:
            assert abs(h[i] - hb) <= 1e-5 * hb
    Mg, Wg = M.cpu().numpy(), _np64(Wp)
    out_rows = fg.astype(bool)
    assert np.array_equal(Wg[out_rows], W64[out_rows]) and Mg[out_rows].sum() == 0
    assert st.n_pruned == (c - n_out) * b // m * n == int(Mg.sum())
    # the pruned rows against the oracle's n:m sweep (alpha does not change them)
    Wo, Mo, _ = O.thanos_nm(W64, None, n, m, B, 0.01, H=H64, alpha=0.0)
    rows = ~out_rows & ~(Mg != Mo).any(axis=1)
    assert rows.sum() >= 0.9 * (c - n_out)
    Wo_cmp = _np64(torch.tensor(Wo).to(torch.bfloat16)) if dtype == "bf16" else Wo
    tol = PU.TOL_W_BF16 if dtype == "bf16" else PU.TOL_W_F32
    assert PU.rel_fro(Wg[rows], Wo_cmp[rows]) <= tol
    if alpha > 0 and np.array_equal(fg, fo):
        Wa, Ma, _ = O.thanos_nm(W64, None, n, m, B, 0.01, H=H64, alpha=alpha)
        assert np.array_equal(Ma[out_rows], Mg[out_rows])
        assert np.array_equal(Wa[out_rows], W64[out_rows])


# ------------------------------------------------------------------------------ bench-size
@pytest.mark.parametrize("c", [4096, 11008], ids=["q_4096x4096", "gate_11008x4096"])
def test_full_size_layer_sampled_rows(T, c):
    """4096-wide bf16 layers of the benchmark (4096 and 11008 rows), B = 128, 50 % unstructured
    and 2:4: structural invariants on the whole output and a float64 replay of sampled rows under
    the GPU's mask."""
    b = 4096
    B = 128
    W = WL.make_weight(c, b, "bf16", seed=2, layer_index=0, device=DEV)
    Xd = WL.make_activations(16384, b, "bf16", "student_t4", 0.005, 0, 50.0, 2, 0, device=DEV)
    H = torch.zeros((b, b), dtype=torch.float32, device=DEV)
    T.hessian_accumulate(H, Xd)
    U, xn = T.prepare_inverse(H, 0.01)
    H64 = _np64(H)
    Hd = O.damped(H64, 0.01)
    xn64 = O.feature_norms(H64)
    rows = np.array([0, 1, 777, 2048, c - 1])
    W64 = _np64(W)
    for mode in ("unstructured", "nm"):
        if mode == "unstructured":
            Wp, M, st = T.prune_layer(W, U, xn, T.UNSTRUCTURED, p=0.5, B=B)
            assert st.n_pruned == c * b // 2 and st.r_left == 0
        else:
            Wp, M, st = T.prune_layer(W, U, xn, T.NM, n=2, m=4, B=B)
            assert bool((M.view(c, b // 4, 4).sum(dim=2) == 2).all())
        assert st.n_blocks == b // B
        assert bool((Wp[M.bool()] == 0).all())
        Mg = M.cpu().numpy()
        # first block: decided on the input weights, so the oracle's mask map applies directly
        if mode == "unstructured":
            S = np.abs(W64) * xn64[None, :]
            r = c * b // 2
            tau = np.partition(S.ravel(), r - 1)[r - 1]
            blk = S[:, :B]
            decided = np.abs(blk - tau) > PU.TIE_REL * tau
            assert np.array_equal(Mg[:, :B][decided], (blk < tau)[decided])
        else:
            Mo_blk = O.nm_block_mask(W64[rows][:, :B], xn64[:B], 2, 4)
            assert np.array_equal(Mg[rows][:, :B], Mo_blk)
        # replay of sampled rows in float64 under the GPU's mask
        Wr = O.replay_rows(W64[rows], Mg[rows], Hd, B)
        Wr = _np64(torch.tensor(Wr).to(torch.bfloat16))
        assert PU.rel_fro(_np64(Wp)[rows], Wr) <= PU.TOL_W_BF16


def test_wide_layer_11008_sampled_rows(T):
    """The down projection of the benchmark at its own shape (4096 x 11008, 86 blocks of 128):
    counts, exact zeros, and a float64 replay of sampled rows under the GPU's mask."""
    c, b, B = 4096, 11008, 128
    W = WL.make_weight(c, b, "bf16", seed=2, layer_index=6, device=DEV)
    Xd = WL.make_activations(12288, b, "bf16", "student_t4", 0.005, 0, 50.0, 2, 3, device=DEV)
    H = torch.zeros((b, b), dtype=torch.float32, device=DEV)
    T.hessian_accumulate(H, Xd)
    U, xn = T.prepare_inverse(H, 0.01)
    Wp, M, st = T.prune_layer(W, U, xn, T.UNSTRUCTURED, p=0.5, B=B)
    assert st.n_pruned == c * b // 2 and st.r_left == 0 and st.n_blocks == b // B
    assert st.select_misses <= 2
    assert bool((Wp[M.bool()] == 0).all())
    Hd = O.damped(_np64(H), 0.01)
    rows = np.array([0, 2047, c - 1])
    Wr = O.replay_rows(_np64(W[rows]), M[rows].cpu().numpy(), Hd, B)
    Wr = _np64(torch.tensor(Wr).to(torch.bfloat16))
    assert PU.rel_fro(_np64(Wp[rows]), Wr) <= PU.TOL_W_BF16


def test_host_buffer_entry_point_matches_device_path(T):
    c, b, a, B = 96, 256, 20000, 64
    W = WL.make_weight(c, b, "bf16", seed=61)
    Xt = _acts(a, b, "bf16", seed=23, mix=0.3)
    Wh, Mh, sth = T.prune_layer_host(W.pin_memory(), Xt.pin_memory(), 0.01, T.UNSTRUCTURED,
                                     p=0.5, B=B)
    H = torch.zeros((b, b), dtype=torch.float32, device=DEV)
    Xd = Xt.to(DEV)
    for t0 in range(0, a, 16384):
        T.hessian_accumulate(H, Xd[t0:t0 + 16384])
    U, xn = T.prepare_inverse(H, 0.01)
    Wp, M, st = T.prune_layer(W.to(DEV), U, xn, T.UNSTRUCTURED, p=0.5, B=B)
    assert sth.n_pruned == st.n_pruned
    same = ~(Mh.numpy() != M.cpu().numpy()).any(axis=1)
    assert same.mean() >= 0.95
    assert PU.rel_fro(_np64(Wh)[same], _np64(Wp)[same]) <= 1e-3


# ------------------------------------------------------------------------------ dense product
@pytest.mark.parametrize("M,N,K,bt", [
    (128, 128, 64, True), (128, 128, 64, False), (300, 520, 128, False), (300, 520, 128, True),
    (64, 72, 8, False), (1000, 4096, 128, False), (257, 132, 200, True), (512, 384, 1024, True),
    # large enough for the CTA-pair kernel (256 x 256 tiles): ragged in M, N and K, the second
    # CTA's half of the last tiles entirely outside the matrix; then a rank-128 update
    (2688, 3712, 264, False), (2688, 3712, 264, True), (8192, 7168, 128, False)])
def test_dense_product_matches_float64(T, M, N, K, bt):
    """The split-bf16 tensor-core product against a float64 product of the same fp32 inputs.
    Bound: a few units of 2^-24 of sum |a||b| per 16-term tensor-core accumulation step."""
    g = torch.Generator().manual_seed(M * 7 + N * 3 + K)
    A = torch.randn((M, K), generator=g) * torch.exp(torch.randn((M, 1), generator=g))
    Bm = torch.randn((N, K) if bt else (K, N), generator=g)
    C0 = torch.randn((M, N), generator=g)
    Ad, Bd = A.to(DEV), Bm.to(DEV)
    want = _np64(A) @ (_np64(Bm).T if bt else _np64(Bm))
    scale = np.abs(_np64(A)) @ np.abs(_np64(Bm).T if bt else _np64(Bm))
    got = _np64(T.dense_product(Ad, Bd, b_transposed=bt))
    assert np.max(np.abs(got - want) / scale) <= 3e-6
    assert np.mean(np.abs(got - want) / scale) <= 4e-7
    # accumulate with a scale factor, into a strided output
    big = torch.zeros((M, N + 8), device=DEV)
    big[:, :N] = C0.to(DEV)
    T.dense_product(Ad, Bd, b_transposed=bt, alpha=-0.5, out=big[:, :N], accumulate=True)
    got2 = _np64(big[:, :N])
    assert np.max(np.abs(got2 - (_np64(C0) - 0.5 * want)) / (scale + np.abs(_np64(C0)))) <= 3e-6
    assert float(big[:, N:].abs().max()) == 0.0


# ------------------------------------------------------------------------------ structured
@pytest.mark.parametrize("c,b,dtype,p,alpha", [
    (96, 256, "f32", 0.3, 0.0), (200, 384, "f32", 0.25, 0.1), (160, 512, "bf16", 0.5, 0.05),
    (64, 136, "f32", 0.1, 0.0), (40, 128, "f32", 0.0, 0.0), (300, 1032, "f32", 0.4, 0.02)])
def test_structured_parity(T, c, b, dtype, p, alpha):
    """Algorithm 2: removed columns, outlier rows and the updated weights against the oracle."""
    W = WL.make_weight(c, b, dtype, seed=91, layer_index=c)
    g = torch.Generator().manual_seed(c + b)
    W = (W.float() * torch.exp(0.7 * torch.randn((c, 1), generator=g))
         * torch.exp(0.5 * torch.randn((1, b), generator=g))).to(W.dtype)
    Xt = WL.make_activations(max(2048, 3 * b), b, dtype, "student_t4", 0.02, 0, 10.0, 31, 0, mix=0.5)
    H = _gpu_hessian(T, Xt)
    H64, W64 = _np64(H), _np64(W)
    U, xn = T.prepare_inverse(H, 0.01)
    Wp, colrm, flags, st = T.prune_layer_structured(W.to(DEV), U, xn, p, alpha,
                                                    H=H if alpha > 0 else None)
    torch.cuda.synchronize()
    Wo, rm_o, out_o, _ = O.thanos_structured(W64, None, p, alpha, 0.01, H=H64)
    s = O.structured_column_count(p, b, alpha)
    rm_g, out_g = colrm.cpu().numpy().astype(bool), flags.cpu().numpy().astype(bool)
    assert rm_g.sum() == s == st.max_s and out_g.sum() == out_o.sum()
    assert st.n_pruned == s * (c - int(out_o.sum()))
    assert np.array_equal(out_g, out_o), "outlier rows differ"
    assert np.array_equal(rm_g, rm_o), "removed columns differ"
    Wg = _np64(Wp)
    assert np.array_equal(Wg[out_g], W64[out_g])                  # outlier rows untouched
    assert np.all(Wg[np.ix_(~out_g, rm_g)] == 0.0)                # exact zeros
    Wo_cmp = _np64(torch.tensor(Wo).to(torch.bfloat16)) if dtype == "bf16" else Wo
    tol = PU.TOL_W_BF16 if dtype == "bf16" else PU.TOL_W_F32
    assert PU.rel_fro(Wg, Wo_cmp) <= tol
    if dtype == "f32" and s:
        # the change of the kept weights itself, not hidden behind the unchanged mass of W
        d_g, d_o = Wg - W64, Wo - W64
        assert PU.rel_fro(d_g[:, ~rm_g], d_o[:, ~rm_g]) <= 2e-4


def test_structured_full_size_sampled_rows(T):
    """4096 x 4096 bf16 layer, 30 % of the columns with 10 % outlier rows: the removed columns are
    the smallest losses of the oracle, and sampled rows match Eq. 8 in float64 for that set."""
    c = b = 4096
    p, alpha = 0.3, 0.1
    W = WL.make_weight(c, b, "bf16", seed=2, layer_index=0, device=DEV)
    Xd = WL.make_activations(16384, b, "bf16", "student_t4", 0.005, 0, 50.0, 2, 0, device=DEV)
    H = torch.zeros((b, b), dtype=torch.float32, device=DEV)
    T.hessian_accumulate(H, Xd)
    U, xn = T.prepare_inverse(H, 0.01)
    Wp, colrm, flags, st = T.prune_layer_structured(W, U, xn, p, alpha, H=H)
    torch.cuda.synchronize()
    H64, W64 = _np64(H), _np64(W)
    s = O.structured_column_count(p, b, alpha)
    rm, outl = colrm.cpu().numpy().astype(bool), flags.cpu().numpy().astype(bool)
    n_out = int(np.ceil(alpha * c - 1e-12))
    assert rm.sum() == s and outl.sum() == n_out and st.n_pruned == s * (c - n_out)
    h = O.row_losses(W64, H=H64)
    sigma, _ = O.outlier_row_order(h, alpha)
    hb = h[sigma[c - n_out]]
    fo = np.zeros(c, dtype=bool)
    fo[sigma[c - n_out:]] = True
    for i in np.nonzero(fo != outl)[0]:
        assert abs(h[i] - hb) <= 1e-5 * hb
    v = O.column_losses(W64[~outl], O.feature_norms(H64))
    vs = np.sort(v)
    lo, hi = vs[s - 1], vs[s]
    assert v[rm].max() <= hi * (1 + 1e-6) and v[~rm].min() >= lo * (1 - 1e-6)
    Wg = _np64(Wp)
    assert np.array_equal(Wg[outl], W64[outl])
    assert bool((Wp[:, colrm.bool()][~flags.bool()] == 0).all())
    rows = np.nonzero(~outl)[0][[0, 1, 1000, 2500, -1]]
    Wr = O.structured_update_rows(W64[rows], rm, O.damped(H64, 0.01))
    Wr = _np64(torch.tensor(Wr).to(torch.bfloat16))
    assert PU.rel_fro(Wg[rows], Wr) <= PU.TOL_W_BF16


def test_structured_edges_and_errors(T):
    """One row, the smallest width, a single removed column; rejected arguments leave the
    context usable."""
    rng = torch.Generator().manual_seed(5)
    for c, b, p in ((1, 8, 0.5), (3, 16, 1.0 / 16), (5, 24, 0.9)):
        X = torch.randn((256, b), generator=rng)
        H = _gpu_hessian(T, X.to(DEV))
        U, xn = T.prepare_inverse(H, 0.01)
        W = torch.randn((c, b), generator=rng).to(DEV)
        Wp, colrm, flags, st = T.prune_layer_structured(W, U, xn, p)
        Wo, rm_o, _, _ = O.thanos_structured(_np64(W), None, p, 0.0, 0.01, H=_np64(H))
        assert np.array_equal(colrm.cpu().numpy().astype(bool), rm_o)
        assert int(flags.sum()) == 0 and st.n_pruned == int(rm_o.sum()) * c
        assert PU.rel_fro(_np64(Wp), Wo) <= PU.TOL_W_F32
    with pytest.raises(T.ThanosError) as e:      # ceil(p b / (1 - alpha)) >= b
        T.prune_layer_structured(W, U, xn, 0.6, alpha=0.5, H=H)
    assert e.value.code == 1
    with pytest.raises(ValueError):              # outlier rows need the Hessian
        T.prune_layer_structured(W, U, xn, 0.25, alpha=0.2)
    with pytest.raises(T.ThanosError) as e:
        T.prune_layer_structured(W, U, xn, 0.25,
                                 workspace=torch.empty(512, dtype=torch.uint8, device=DEV))
    assert e.value.code == 5
    Wp, colrm, flags, st = T.prune_layer_structured(W, U, xn, 0.25)
    assert st.status == 0 and int(colrm.sum()) == 6


# ------------------------------------------------------------------------------ config shapes
@pytest.mark.parametrize("layer", [0, 4], ids=["q_768x768", "fc1_3072x768"])
def test_opt125m_layer_shapes_full_oracle(T, layer):
    """The 768-wide OPT-125M-shaped layers (2:4, B = 128, fp32) against the oracle's whole sweep,
    with the Hessian from 8192 of the configuration's tokens.  The 3072-wide layer of the set is
    stepped beside the oracle block by block in
    test_gpu_fullsize.py::test_state_drift_of_the_fp32_sweep_is_what_flips_masks."""
    cfg = WL.CONFIGS["opt125m"]
    L = cfg.layers[layer]
    W = WL.config_weight(cfg, layer)
    Xt = WL.config_activations(cfg, L.input_id, L.b, a=8192)
    H = _gpu_hessian(T, Xt, chunks=2)
    out = _check_sweep(T, W, H, "nm", 0.0, cfg.n, cfg.m, cfg.B, cfg.damp_rel, PU.TOL_W_F32)
    assert out["mismatch"] <= 4


@pytest.mark.parametrize("mode,c", [("nm", 28672), ("unstructured", 8192)],
                         ids=["gate_28672x8192_2of4", "q_8192x8192_unstr60"])
def test_llama2_70b_width_8192_full_shapes(T, mode, c):
    """The 8192-wide layers of the LLaMA-2-70B-shaped set at their own shapes (28672 x 8192 with
    2:4, 8192 x 8192 with 60 % unstructured, B = 128, bf16): counts, exact zeros, and a float64
    replay of sampled rows under the GPU's mask."""
    cfg = WL.CONFIGS["llama2_70b"]
    b, B = 8192, cfg.B
    W = WL.make_weight(c, b, "bf16", seed=cfg.seed, layer_index=0, device=DEV)
    Xd = WL.config_activations(cfg, 0, b, device=DEV, a=12288)
    H = torch.zeros((b, b), dtype=torch.float32, device=DEV)
    T.hessian_accumulate(H, Xd)
    del Xd
    U, xn = T.prepare_inverse(H, cfg.damp_rel)
    if mode == "nm":
        Wp, M, st = T.prune_layer(W, U, xn, T.NM, n=2, m=4, B=B)
        assert bool((M.view(c, b // 4, 4).sum(dim=2) == 2).all())
        assert st.n_pruned == c * b // 2
    else:
        Wp, M, st = T.prune_layer(W, U, xn, T.UNSTRUCTURED, p=0.6, B=B)
        assert st.n_pruned == PU.expected_removed(0.6, c, b) and st.r_left == 0
        assert st.select_misses <= 2
    assert st.n_blocks == b // B and bool((Wp[M.bool()] == 0).all())
    Hd = O.damped(_np64(H), cfg.damp_rel)
    rows = torch.tensor([0, c // 3, c - 1], device=DEV)
    Wr = O.replay_rows(_np64(W[rows]), M[rows].cpu().numpy(), Hd, B)
    Wr = _np64(torch.tensor(Wr).to(torch.bfloat16))
    assert PU.rel_fro(_np64(Wp[rows]), Wr) <= PU.TOL_W_BF16


def test_llama3_8b_gate_projection_full_shape(T):
    """14336 x 4096 (gate / up of the LLaMA-3-8B-shaped set), 4:8, B = 256, bf16, all rows: the
    CTA-per-row solve at its real row count; pattern, zeros, sampled float64 replay."""
    cfg = WL.CONFIGS["llama3_8b"]
    c, b, B = 14336, 4096, cfg.B
    W = WL.make_weight(c, b, "bf16", seed=cfg.seed, layer_index=4, device=DEV)
    Xd = WL.config_activations(cfg, 2, b, device=DEV, a=16384)
    H = torch.zeros((b, b), dtype=torch.float32, device=DEV)
    T.hessian_accumulate(H, Xd)
    del Xd
    U, xn = T.prepare_inverse(H, cfg.damp_rel)
    Wp, M, st = T.prune_layer(W, U, xn, T.NM, n=cfg.n, m=cfg.m, B=B)
    assert bool((M.view(c, b // 8, 8).sum(dim=2) == 4).all())
    assert st.n_pruned == c * b // 2 and st.n_blocks == b // B and st.max_s == B // 2
    assert bool((Wp[M.bool()] == 0).all())
    Hd = O.damped(_np64(H), cfg.damp_rel)
    rows = torch.tensor([0, 5000, c - 1], device=DEV)
    Wr = O.replay_rows(_np64(W[rows]), M[rows].cpu().numpy(), Hd, B)
    Wr = _np64(torch.tensor(Wr).to(torch.bfloat16))
    assert PU.rel_fro(_np64(Wp[rows]), Wr) <= PU.TOL_W_BF16


def test_threshold_jumps_between_blocks(T):
    """Column blocks of very different scale move the global threshold by far more than the
    bracket window from one block to the next: the bracket misses, the radix passes take over
    (and the window stays wide for the rest of the sweep); the result is still the oracle's."""
    c, b, B = 96, 768, 64
    W = WL.make_weight(c, b, "f32", seed=97)
    g = torch.Generator().manual_seed(11)
    blk_scale = torch.tensor([1.0, 30.0, 0.05, 8.0, 0.3, 100.0, 1.0, 0.01, 3.0, 50.0, 0.2, 5.0])
    W = W * blk_scale.repeat_interleave(B)[None, :]
    Xt = WL.make_activations(4096, b, "f32", "normal", 0.0, 0, 1.0, 23, 0, mix=0.4)
    H = _gpu_hessian(T, Xt)
    out = _check_sweep(T, W, H, "unstructured", 0.5, 0, 0, B, 0.01, PU.TOL_W_F32)
    assert out["stats"].select_misses >= 1
