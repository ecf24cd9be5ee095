"""Comparison helpers for the CUDA-vs-oracle parity tests (no method arithmetic beyond the
metric formula needed to classify near-ties)."""

from __future__ import annotations

import math

import numpy as np

# Tolerances of the parity protocol: H relative Frobenius, pruned weights relative Frobenius
# (fp32 / bf16 inputs), and the relative score gap under which a mask difference is a near-tie.
TOL_H = 1e-5
TOL_W_F32 = 1e-3
TOL_W_BF16 = 5e-3
TIE_REL = 1e-6


def rel_fro(a, b) -> float:
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    d = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / (d if d > 0 else 1.0))


def block_threshold(W_before, xnorm, j1, mask_block_oracle, r_before):
    """Score of the r-th smallest residual entry (the block threshold) in float64."""
    S = np.abs(W_before[:, j1:]) * xnorm[None, j1:]
    if r_before <= 0:
        return -1.0, S
    return float(np.partition(S.ravel(), r_before - 1)[r_before - 1]), S


def classify_unstructured_block(mask_gpu_blk, mask_or_blk, S_blk, tau, tie_rel=None):
    """Split mask differences of one block into near-ties (oracle score within TIE_REL of the
    block threshold, relative) and real mismatches.  Returns (n_near_tie, n_bad)."""
    diff = mask_gpu_blk != mask_or_blk
    if not diff.any():
        return 0, 0
    s = S_blk[diff]
    tie_rel = TIE_REL if tie_rel is None else tie_rel
    near = np.abs(s - tau) <= tie_rel * max(tau, 1e-300)
    return int(near.sum()), int((~near).sum())


def classify_nm_block(mask_gpu_blk, mask_or_blk, S_blk, n, m, tie_rel=None):
    """n:m: a difference inside a group is a near-tie if the group's n-th and (n+1)-th smallest
    oracle scores are within TIE_REL (relative)."""
    c, w = S_blk.shape
    near = bad = 0
    diff = mask_gpu_blk != mask_or_blk
    rows, cols = np.nonzero(diff)
    seen = set()
    for i, j in zip(rows, cols):
        g = j // m
        if (i, g) in seen:
            continue
        seen.add((i, g))
        s = np.sort(S_blk[i, g * m:(g + 1) * m])
        gap = abs(s[n] - s[n - 1])
        cnt = int(diff[i, g * m:(g + 1) * m].sum())
        if gap <= (TIE_REL if tie_rel is None else tie_rel) * max(s[n], 1e-300):
            near += cnt
        else:
            bad += cnt
    return near, bad


def expected_removed(p, c, b) -> int:
    return int(math.floor(p * c * b))
