"""GPU parity at the sizes, launch shapes and select routes the benchmark configurations take.

The whole-sweep oracle is too slow for these shapes, so every test here combines checks that stay
cheap at any size:

* the selection function of Algorithm 1 (Eq. psi with the running budget) applied in float64 to
  the GPU's OWN pre-block state, block by block (the sweep is stepped through
  thanos_prune_block with its statistics carried over, which takes the same bracket + refine
  route as thanos_prune_layer);
* a float64 replay of sampled rows under the GPU's mask (Eq. 8 per block);
* block steps from a given state against the literal row update of Eqs. 5-8 (late blocks) and
  against its optimality condition (first block: the gradient of the row objective vanishes on
  every weight that is not removed);
* the defining identity of the factor, U H_d U^T = I, on sampled rows in float64.
"""

import math

import numpy as np
import pytest
import torch

import workloads as WL
from oracle import thanos_oracle as O
from tests import parity_utils as PU

pytestmark = pytest.mark.gpu

DEV = "cuda"


@pytest.fixture(scope="module")
def T():
    import paper_2504_05346_b200 as T_
    from paper_2504_05346_b200 import build as B_

    B_.build()
    T_.load_library()
    return T_


def _np64(t):
    return t.detach().cpu().double().numpy()


def _hessian(T, Xd):
    b = Xd.shape[1]
    H = torch.zeros((b, b), dtype=torch.float32, device=DEV)
    ws = torch.empty(max(256, T.workspace_bytes(0, 0, b, 0, T.BF16 if Xd.dtype == torch.bfloat16
                                                else T.F32)), dtype=torch.uint8, device=DEV)
    T.hessian_accumulate(H, Xd, workspace=ws, check=True)
    return H


def _stats(T, st):
    return T.PruneStats.from_bytes(bytes(st.cpu().numpy().tobytes()))


def step_sweep(T, Wc, U, xn, mode, n, m, B, r0, on_block=None, workspace=None):
    """The sweep one block at a time through thanos_prune_block, in place on the fp32 working
    weights `Wc`; the budget and the statistics are carried from call to call.  `on_block(j1, j2,
    r_before, before, mask)` gets a device copy of the residual `Wc[:, j1:]` taken before the step
    (only when `wants(j1)` says so) and the device mask after it."""
    c, b = Wc.shape
    mask = torch.zeros((c, b), dtype=torch.uint8, device=DEV)
    stats = torch.zeros(64, dtype=torch.uint8, device=DEV)
    r = torch.tensor([r0], dtype=torch.int64, device=DEV)
    if workspace is None:
        workspace = torch.empty(T.workspace_bytes(2, c, b, B, T.F32), dtype=torch.uint8, device=DEV)
    for j1 in range(0, b, B):
        j2 = min(b, j1 + B)
        r_before = int(r.item()) if mode == T.UNSTRUCTURED else 0
        before = None
        if on_block is not None and on_block.wants(j1):
            before = Wc[:, j1:].clone()
        T.prune_block(Wc, mask, U, xn, mode, n, m, B, j1, r if mode == T.UNSTRUCTURED else None,
                      stats, workspace=workspace)
        if before is not None:
            on_block(j1, j2, r_before, before, mask)
    torch.cuda.synchronize()
    return mask, _stats(T, stats), (int(r.item()) if mode == T.UNSTRUCTURED else 0)


class PsiOnOwnState:
    """Per block: the float64 threshold of Eq. psi on the GPU's own pre-block weights against the
    mask the GPU wrote.  Entries whose score is within TIE_REL (relative) of the threshold may go
    either way; every other entry of the block must be removed iff its score is below it."""

    def __init__(self, xn64, every=1, full_psi_blocks=()):
        self.xn = xn64
        self.every = every
        self.full = set(full_psi_blocks)
        self.near = 0
        self.blocks = 0
        self.max_tie_gap = 0.0

    def wants(self, j1):
        return True if self.every == 1 else ((j1 // self._B) % self.every == 0)

    def bind(self, B):
        self._B = B
        return self

    def __call__(self, j1, j2, r_before, before, mask):
        Wb = _np64(before)
        Mg = mask[:, j1:j2].cpu().numpy()
        S = O.metric(Wb, self.xn[j1:])
        w = j2 - j1
        blk = S[:, :w]
        if r_before <= 0:
            assert Mg.sum() == 0
            return
        tau = float(np.partition(S.ravel(), r_before - 1)[r_before - 1])  # r-th smallest score
        decided = np.abs(blk - tau) > PU.TIE_REL * tau
        want = blk < tau
        bad = int((Mg.astype(bool) != want)[decided].sum())
        assert bad == 0, "block at %d: %d entries on the wrong side of the threshold" % (j1, bad)
        und = ~decided
        flips = und & (Mg.astype(bool) != (blk <= tau))
        self.near += int(und.sum())
        if flips.any():
            self.max_tie_gap = max(self.max_tie_gap, float(np.max(np.abs(blk[flips] - tau)) / tau))
        # the count removed in the block is fixed by the threshold up to the undecided entries
        lo, hi = int((want & decided).sum()), int((want & decided).sum() + und.sum())
        assert lo <= int(Mg.sum()) <= hi
        if (j1 // self._B) in self.full:
            Mo = O.psi(Wb, self.xn[j1:], r_before)[:, :w]
            near, bad = PU.classify_unstructured_block(Mg, Mo, blk, tau)
            assert bad == 0
        self.blocks += 1


# ------------------------------------------------------------------------------ select, full size
def test_select_is_psi_on_every_block_of_a_benchmark_layer(T):
    """4096 x 4096 bf16, 50 % unstructured, B = 128 (the benchmark's attention projections): all
    32 blocks, 31 of them through the bracket + refine route, against Eq. psi on the same state;
    the stepped sweep is then the one-call sweep bit for bit, and sampled rows match a float64
    replay under the GPU's mask before any rounding (weights and the update itself)."""
    c = b = 4096
    B = 128
    W = WL.make_weight(c, b, "bf16", seed=2, layer_index=0, device=DEV)
    Xd = WL.make_activations(16384, b, "bf16", "student_t4", 0.005, 0, 50.0, 2, 0, device=DEV)
    H = _hessian(T, Xd)
    del Xd
    U, xn = T.prepare_inverse(H, 0.01)
    H64 = _np64(H)
    xn64 = O.feature_norms(H64)
    Wp, M, st = T.prune_layer(W, U, xn, T.UNSTRUCTURED, p=0.5, B=B)
    Wc = W.float().contiguous()
    chk = PsiOnOwnState(xn64, full_psi_blocks=(1, 31)).bind(B)
    Ms, sts, r_left = step_sweep(T, Wc, U, xn, T.UNSTRUCTURED, 0, 0, B, c * b // 2, chk)
    assert chk.blocks == b // B and r_left == 0 and sts.n_pruned == c * b // 2
    assert sts.select_misses == 0 == st.select_misses      # every later block: bracket + refine
    assert sts.select_rescans == 0
    assert torch.equal(Ms, M)
    assert torch.equal(Wc.to(torch.bfloat16), Wp)
    print("near-tie entries %d, largest relative gap of an undecided flip %.2e"
          % (chk.near, chk.max_tie_gap))
    # float64 replay of sampled rows under this mask, compared BEFORE the final rounding
    rows = np.array([0, 1, 777, 2048, c - 1])
    W64 = _np64(W)[rows]
    Mg = Ms.cpu().numpy()[rows]
    Wr = O.replay_rows(W64, Mg, O.damped(H64, 0.01), B)
    Wg = _np64(Wc)[rows]
    assert PU.rel_fro(Wg, Wr) <= PU.TOL_W_F32
    Dg, Dr = Wg - (1 - Mg) * W64, Wr - (1 - Mg) * W64
    assert PU.rel_fro(Dg, Dr) <= 2e-3


def test_select_overflow_routes_with_exact_ties(T):
    """Weights on a three-level grid and a diagonal Hessian: 40 % of all scores are the SAME number,
    and the block threshold sits inside that plateau.  The bracket window then holds far more keys
    than one CTA (6144) or the global list (c b / 8) can copy out, so the refining pass rescans the
    residual, and the plateau is split by the (row, column) order.  With a diagonal Hessian no
    kept weight changes, so everything is exact integer work: masks and weights must equal the
    oracle's bit for bit."""
    c, b, B = 4096, 2560, 128
    g = torch.Generator().manual_seed(5)
    lev = torch.tensor([0.01, 0.02, 0.03])
    idx = torch.multinomial(torch.tensor([0.3, 0.4, 0.3]), c * b, replacement=True, generator=g)
    sgn = torch.randint(0, 2, (c * b,), generator=g).float() * 2 - 1
    W = (lev[idx] * sgn).reshape(c, b).contiguous()
    H = (2.0 * 4096.0) * torch.eye(b, dtype=torch.float32)
    U, xn = T.prepare_inverse(H.to(DEV), 0.01)
    Wp, M, st = T.prune_layer(W.to(DEV), U, xn, T.UNSTRUCTURED, p=0.5, B=B)
    assert st.n_pruned == c * b // 2 and st.r_left == 0 and st.n_blocks == b // B
    assert st.select_rescans >= 10, st       # per-CTA overflow early, global overflow later
    assert st.n_tied > 0
    Wo, Mo, _ = O.thanos_unstructured_fast(_np64(W), None, 0.5, B, 0.01, H=_np64(H))
    assert np.array_equal(M.cpu().numpy(), Mo)
    assert np.array_equal(_np64(Wp), Wo)
    assert np.array_equal(Wo, _np64(W) * (1 - Mo))      # nothing but the removals changed


# ------------------------------------------------------------------------------ Hessian, bench call
def test_hessian_one_call_of_the_benchmark_length(T):
    """One thanos_hessian_accumulate call over 262144 tokens at b = 4096 (the launch the benchmark
    issues: 16 k - 64 k tokens per slice, several slices per tile): sampled entries against float64
    dot products, the call's device status word, symmetry."""
    b, a = 4096, 262144
    Xd = WL.make_activations(a, b, "bf16", "student_t4", 0.005, 0, 50.0, 2, 0, device=DEV)
    H = _hessian(T, Xd)
    torch.cuda.synchronize()
    rng = np.random.default_rng(1)
    ii = rng.integers(0, b, 40)
    jj = rng.integers(0, b, 40)
    ii[:8] = jj[:8]
    outl = WL.outlier_channels(b, 0.005, 0, 2, 0).numpy()
    ii[8:12] = outl[:4]
    jj[12:14] = outl[4:6]
    ii[14], jj[14] = 0, b - 1
    ii[15], jj[15] = b - 1, 0
    cols = np.unique(np.concatenate([ii, jj]))
    Xc = _np64(Xd[:, torch.as_tensor(cols, device=DEV)])
    pos = {c_: k for k, c_ in enumerate(cols)}
    Ho = O.hessian(Xc.T)                       # float64 Hessian of the sampled features
    Hs = _np64(H[torch.as_tensor(ii, device=DEV), torch.as_tensor(jj, device=DEV)])
    want = np.array([Ho[pos[i], pos[j]] for i, j in zip(ii, jj)])
    scale = np.sqrt(np.array([Ho[pos[i], pos[i]] * Ho[pos[j], pos[j]] for i, j in zip(ii, jj)]))
    assert np.max(np.abs(Hs - want) / scale) <= 1e-5
    assert bool(torch.isfinite(H).all())
    assert float((H - H.T).abs().max()) <= 1e-5 * float(H.abs().max())


# ------------------------------------------------------------------------------ wide layers
def _rows_times_matrix(rows64, M32, add_diag=0.0, chunk=2048, absolute=False):
    """rows64 [k, n] (float64) times the fp32 matrix M32 [n, n] (a host tensor) + add_diag * rows64,
    in float64, converting M32 a column strip at a time (`absolute`: of the absolute values)."""
    n = M32.shape[0]
    out = np.empty((rows64.shape[0], n))
    for c0 in range(0, n, chunk):
        c1 = min(n, c0 + chunk)
        strip = M32[:, c0:c1].double().numpy()
        out[:, c0:c1] = rows64 @ (np.abs(strip) if absolute else strip)
    return out + add_diag * rows64


def _factor_identity_error(U32, H32, lam, rows):
    """max |(U H_d U^T - I)[rows, :]| in float64 (U, H host fp32 tensors, H_d = H + lam I)."""
    Ur = U32[rows].double().numpy()
    Tm = _rows_times_matrix(Ur, H32, add_diag=lam)            # U[rows] H_d
    n = U32.shape[0]
    worst = 0.0
    for r0 in range(0, n, 2048):
        r1 = min(n, r0 + 2048)
        E = Tm @ U32[r0:r1].double().numpy().T                # columns r0..r1 of U[rows] H_d U^T
        for k, i in enumerate(rows):
            if r0 <= i < r1:
                E[k, i - r0] -= 1.0
        worst = max(worst, float(np.max(np.abs(E))))
    return worst


def _kkt_first_block(T, W, U, xn, H32, lam, mode, n, m, B, r0, rows):
    """One block step at j1 = 0 from the state W: for sampled rows the change delta of the WHOLE row
    must satisfy the optimality condition of Eq. 8 -- delta_q = -w_q, and the gradient delta H_d
    vanishes on every weight that is not removed (it is carried by the removed positions only)."""
    c, b = W.shape
    Wc = W.float().contiguous()
    mask = torch.zeros((c, b), dtype=torch.uint8, device=DEV)
    stats = torch.zeros(64, dtype=torch.uint8, device=DEV)
    r = torch.tensor([r0], dtype=torch.int64, device=DEV)
    T.prune_block(Wc, mask, U, xn, mode, n, m, B, 0, r if mode == T.UNSTRUCTURED else None, stats)
    torch.cuda.synchronize()
    delta = _np64(Wc[rows]) - _np64(W[rows])
    Mq = mask[rows].cpu().numpy().astype(bool)
    assert not Mq[:, B:].any()
    g = _rows_times_matrix(delta, H32, add_diag=lam)
    # g_j is a sum with heavy cancellation (columns of high-energy features carry terms 1e3 times
    # the result): its natural scale is sum_i |delta_i| |H_d[i, j]|
    scale = _rows_times_matrix(np.abs(delta), H32, add_diag=lam, absolute=True)
    worst = 0.0
    for k in range(len(rows)):
        q = Mq[k]
        if not q.any():
            assert not delta[k].any()
            continue
        assert np.array_equal(delta[k][q], -_np64(W[rows[k]])[q])
        worst = max(worst, float(np.max(np.abs(g[k][~q]) / scale[k][~q])))
        # the check has teeth: on the removed positions the gradient is far from cancelling
        assert np.max(np.abs(g[k][q]) / scale[k][q]) >= 1e-2
    print("first block, b = %d: largest |delta H_d| / (|delta| |H_d|) on kept weights %.2e" % (b, worst))
    assert worst <= 1e-4
    return mask


def _late_block_literal(T, W, U, xn, H32, lam, mode_nm, B, j1, rows):
    """One n:m block step at a late j1 from the state W against the LITERAL update of Eqs. 5-8
    with the float64 inverse of the residual Hessian H_d[j1:, j1:]."""
    n, m = mode_nm
    c, b = W.shape
    Wc = W.float().contiguous()
    mask = torch.zeros((c, b), dtype=torch.uint8, device=DEV)
    stats = torch.zeros(64, dtype=torch.uint8, device=DEV)
    T.prune_block(Wc, mask, U, xn, T.NM, n, m, B, j1, None, stats)
    torch.cuda.synchronize()
    Hres = H32[j1:, j1:].double().numpy() + lam * np.eye(b - j1)
    Hinv = np.linalg.inv(Hres)
    xn64 = O.feature_norms(H32[j1:, j1:].double().numpy())
    j2 = min(b, j1 + B)
    W64 = _np64(W[rows])[:, j1:]
    Mo = O.nm_block_mask(W64[:, : j2 - j1], xn64[: j2 - j1], n, m)
    Mg = mask[rows][:, j1:j2].cpu().numpy()
    assert np.array_equal(Mg, Mo)
    Wg = _np64(Wc[rows])[:, j1:]
    for k in range(len(rows)):
        q = O.phi(Mo[k])
        delta, _ = O.row_update(Hinv, q, W64[k])
        want = W64[k] + delta
        want[q] = 0.0
        assert PU.rel_fro(Wg[k], want) <= 1e-4
        dg = Wg[k] - W64[k]
        assert PU.rel_fro(dg, want - W64[k]) <= 2e-3
    assert torch.equal(Wc[:, :j1], W.float()[:, :j1])


@pytest.mark.parametrize("b", [8200, 11008])
def test_factor_identity_on_grouped_panels_and_cta_pairs(T, b):
    """Widths whose factorisation runs its large products on CTA pairs (256 x 256 tiles) with the
    panels in groups of four: 11008 (the benchmark's widest layer: 86 panels = 21 groups and two
    left over) and 8200 (a ragged last panel of 8 columns, ragged 256-tiles in every product).
    U is upper-triangular and U H_d U^T = I on sampled rows in float64."""
    Xd = WL.make_activations(2 * b, b, "bf16", "student_t4", 0.005, 0, 50.0, 5, 1, device=DEV)
    H = _hessian(T, Xd)
    del Xd
    U, xn = T.prepare_inverse(H, 0.01)
    assert bool((torch.tril(U, -1) == 0).all()) and bool(torch.isfinite(U).all())
    H32, U32 = H.cpu(), U.cpu()
    lam = 0.01 * float(np.mean(np.diag(H32.numpy()).astype(np.float64)))
    err = _factor_identity_error(U32, H32, lam, [0, 1, b // 2 + 3, b - 130, b - 1])
    print("max |U H_d U^T - I| on sampled rows, b = %d: %.2e" % (b, err))
    assert err <= 1e-4
    assert np.allclose(_np64(xn), O.feature_norms(_np64(H)), rtol=1e-6)


def test_llama3_8b_down_projection_width(T):
    """b = 14336 (the down projection of the LLaMA-3-8B-shaped set), 4:8, B = 256, 256 rows:
    n:m pattern and exact zeros on the whole output, the factor's defining identity on sampled
    rows, a late block step against the literal Eqs. 5-8, the first block step against the
    optimality condition, and a float64 replay is left to the narrower layers (its float64 factor
    of a 14336 x 14336 matrix alone takes minutes on the host)."""
    cfg = WL.CONFIGS["llama3_8b"]
    c, b, B = 256, 14336, cfg.B
    W = WL.make_weight(c, b, "bf16", seed=cfg.seed, layer_index=6, device=DEV)
    Xd = WL.config_activations(cfg, 3, b, device=DEV, a=16384)
    H = _hessian(T, Xd)
    del Xd
    U, xn = T.prepare_inverse(H, cfg.damp_rel)
    Wp, M, st = T.prune_layer(W, U, xn, T.NM, n=cfg.n, m=cfg.m, B=B)
    assert st.n_blocks == b // B and st.n_pruned == c * b // 2 and st.max_s == B // 2
    assert bool((M.view(c, b // 8, 8).sum(dim=2) == 4).all())
    assert bool((Wp[M.bool()] == 0).all()) and bool(torch.isfinite(Wp.float()).all())
    H32, U32 = H.cpu(), U.cpu()
    lam = cfg.damp_rel * float(np.mean(np.diag(H32.numpy()).astype(np.float64)))
    err = _factor_identity_error(U32, H32, lam, [0, 5000, b - 1])
    print("max |U H_d U^T - I| on sampled rows, b = %d: %.2e" % (b, err))
    assert err <= 1e-4
    rows = [0, 100, c - 1]
    _late_block_literal(T, W, U, xn, H32, lam, (cfg.n, cfg.m), B, b - 2048, rows)
    _kkt_first_block(T, W, U, xn, H32, lam, T.NM, cfg.n, cfg.m, B, 0, rows)


@pytest.mark.parametrize("mode", ["nm", "unstructured"])
def test_llama2_70b_down_projection_width(T, mode):
    """b = 28672 (the down projection of the LLaMA-2-70B-shaped set: 224 blocks, H and U of
    3.3 GB each in fp32), B = 128, 512 rows, 2:4 and 60 % unstructured."""
    cfg = WL.CONFIGS["llama2_70b"]
    c, b, B = 512, 28672, cfg.B
    W = WL.make_weight(c, b, "bf16", seed=cfg.seed, layer_index=3, device=DEV)
    Xd = WL.config_activations(cfg, 2, b, device=DEV, a=12288)
    H = _hessian(T, Xd)
    del Xd
    U, xn = T.prepare_inverse(H, cfg.damp_rel)
    H32 = H.cpu()
    lam = cfg.damp_rel * float(np.mean(np.diag(H32.numpy()).astype(np.float64)))
    rows = [0, 255, c - 1]
    if mode == "nm":
        Wp, M, st = T.prune_layer(W, U, xn, T.NM, n=2, m=4, B=B)
        assert bool((M.view(c, b // 4, 4).sum(dim=2) == 2).all()) and st.max_s == B // 2
        U32 = U.cpu()
        err = _factor_identity_error(U32, H32, lam, [0, 9999, b - 1])
        print("max |U H_d U^T - I| on sampled rows, b = %d: %.2e" % (b, err))
        assert err <= 1e-4
        del U32
        _late_block_literal(T, W, U, xn, H32, lam, (2, 4), B, b - 2048, rows)
        _kkt_first_block(T, W, U, xn, H32, lam, T.NM, 2, 4, B, 0, rows)
    else:
        r0 = PU.expected_removed(0.6, c, b)
        Wp, M, st = T.prune_layer(W, U, xn, T.UNSTRUCTURED, p=0.6, B=B)
        assert st.n_pruned == r0 and st.r_left == 0 and st.select_misses <= 2
        # the stepped sweep with Eq. psi on its own state at every eighth block, then the same
        # result as the one-call sweep
        xn64 = np.concatenate([O.feature_norms(H32[k:k + 2048, k:k + 2048].double().numpy())
                               for k in range(0, b, 2048)])
        Wc = W.float().contiguous()
        chk = PsiOnOwnState(xn64, every=8).bind(B)
        Ms, sts, r_left = step_sweep(T, Wc, U, xn, T.UNSTRUCTURED, 0, 0, B, r0, chk)
        assert chk.blocks == b // B // 8 and r_left == 0
        assert torch.equal(Ms, M) and torch.equal(Wc.to(torch.bfloat16), Wp)
        _kkt_first_block(T, W, U, xn, H32, lam, T.UNSTRUCTURED, 0, 0, B, r0, rows)
    assert st.n_blocks == b // B
    assert bool((Wp[M.bool()] == 0).all()) and bool(torch.isfinite(Wp.float()).all())


# ------------------------------------------------------------------------------ drift of the state
def _oracle_states(W64, H64, n, m, B, damp):
    """The oracle's n:m sweep block by block (one factorisation, Eqs. 5-8 per block), yielding the
    state before each block and the block's mask."""
    Wc = W64.copy()
    U = O.inverse_factor(O.damped(H64, damp))
    xn = O.feature_norms(H64)
    b = W64.shape[1]
    for j1 in range(0, b, B):
        j2 = min(b, j1 + B)
        Mb = O.nm_block_mask(Wc[:, j1:j2], xn[j1:j2], n, m)
        yield j1, j2, Wc, Mb
        O.block_update_from_factor(Wc, Mb, U, j1, j2)


@pytest.mark.parametrize("name,c,b,a,dtype,n,m,B,cfgname,layer", [
    ("opt125m_fc2", 768, 3072, 8192, "f32", 2, 4, 128, "opt125m", 5),
    ("llama3_like_4of8_b256", 192, 4096, 8192, "bf16", 4, 8, 256, "llama3_8b", 0),
])
def test_state_drift_of_the_fp32_sweep_is_what_flips_masks(T, name, c, b, a, dtype, n, m, B,
                                                           cfgname, layer):
    """Deep into a wide layer the fp32 working weights (and the fp32 factor behind every update)
    differ from the float64 oracle's by about 1e-5, so a group whose two competing scores are closer
    than that can be decided differently although each side applies the n:m rule of Algorithm 4
    correctly to its own numbers.  The GPU's sweep is stepped beside the oracle's; per block and on
    the rows whose masks agreed so far: (1) the GPU's mask is the n:m rule on the GPU's own state
    (1e-6 near-ties aside), (2) every group decided differently from the oracle has an oracle gap no
    larger than the two sides' score differences in that group (so the drift, not the selection,
    explains it), (3) the relative state difference stays below 1e-4.  The largest gap of a flip
    and the drift are printed: they are the achieved tie bound of this configuration."""
    cfg = WL.CONFIGS[cfgname]
    L = cfg.layers[layer]
    W = WL.make_weight(c, b, dtype, cfg.seed, layer)
    Xt = WL.config_activations(cfg, L.input_id, b, a=a)
    H = _hessian(T, Xt.to(DEV))
    U, xn = T.prepare_inverse(H, cfg.damp_rel)
    H64, W64 = _np64(H), _np64(W)
    xn64 = O.feature_norms(H64)
    Wc = W.to(DEV).float().contiguous()
    mask = torch.zeros((c, b), dtype=torch.uint8, device=DEV)
    stats = torch.zeros(64, dtype=torch.uint8, device=DEV)
    ws = torch.empty(T.workspace_bytes(2, c, b, B, T.F32), dtype=torch.uint8, device=DEV)
    clean = np.ones(c, dtype=bool)
    drift_max = gap_max = 0.0
    flips = nears = 0
    for j1, j2, Wo_before, Mo in _oracle_states(W64, H64, n, m, B, cfg.damp_rel):
        Wg_before = _np64(Wc[:, j1:])
        T.prune_block(Wc, mask, U, xn, T.NM, n, m, B, j1, None, stats, workspace=ws)
        Mg = mask[:, j1:j2].cpu().numpy()
        w = j2 - j1
        Sg = O.metric(Wg_before[:, :w], xn64[j1:j2])
        So = O.metric(Wo_before[:, j1:j2], xn64[j1:j2])
        # (1) the GPU's mask against the rule on its own state
        near, bad = PU.classify_nm_block(Mg, O.nm_block_mask(Wg_before[:, :w], xn64[j1:j2], n, m),
                                         Sg, n, m)
        assert bad == 0
        nears += near
        # (3) state difference on the clean rows, whole residual
        if clean.any():
            drift_max = max(drift_max, PU.rel_fro(Wg_before[clean], Wo_before[clean][:, j1:]))
        # (2) groups decided differently from the oracle
        diff = (Mg != Mo) & clean[:, None]
        for i, g in {(i, j // m) for i, j in zip(*np.nonzero(diff))}:
            so = np.sort(So[i, g * m:(g + 1) * m])
            gap = (so[n] - so[n - 1]) / so[n]
            e = np.max(np.abs(Sg[i, g * m:(g + 1) * m] - So[i, g * m:(g + 1) * m])) / so[n]
            assert gap <= 2.0 * e + PU.TIE_REL, (j1, i, g, gap, e)
            gap_max = max(gap_max, gap)
            flips += 1
        clean &= ~(Mg != Mo).any(axis=1)
    torch.cuda.synchronize()
    print("%s: %d groups decided differently (largest oracle gap %.2e), %d near-tie entries on the "
          "GPU's own state, largest relative state difference %.2e, rows still identical %d of %d"
          % (name, flips, gap_max, nears, drift_max, int(clean.sum()), c))
    assert drift_max <= 1e-4
    assert flips <= max(4, c * b // m // 50000)
    assert clean.sum() >= 0.97 * c
    # the final weights of the rows that followed the oracle's masks throughout (the generator
    # updates its state in place, so after its last step `Wo_before` is the oracle's result)
    assert PU.rel_fro(_np64(Wc)[clean], Wo_before[clean]) <= PU.TOL_W_F32
