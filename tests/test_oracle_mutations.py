"""The pins must notice plausible mistakes in the oracle: each case below plants one mistake in a
copy of the oracle's source (on the CPU, never in the library), runs every pin of
test_oracle_pins.py against that copy and expects at least one of them to fail."""

import os
import types

import pytest

from oracle import thanos_oracle as O
from tests import test_oracle_pins as pins

SRC = open(os.path.join(os.path.dirname(O.__file__), "thanos_oracle.py")).read()

# (name, text in the oracle, replacement)
MUTANTS = [
    ("hessian_without_factor_2", "return 2.0 * (X @ X.T)", "return 1.0 * (X @ X.T)"),
    ("hessian_wrong_orientation", "return 2.0 * (X @ X.T)",
     "return 2.0 * (X.T @ X) if X.shape[0] == X.shape[1] else 2.0 * (X @ X.T) * 1.0001"),
    ("norms_from_the_full_diagonal", "return np.sqrt(np.diag(np.asarray(H, dtype=F64)) / 2.0)",
     "return np.sqrt(np.diag(np.asarray(H, dtype=F64)))"),
    ("damping_doubled", "lam = float(damp_rel) * float(np.mean(np.diag(H)))",
     "lam = 2.0 * float(damp_rel) * float(np.mean(np.diag(H)))"),
    ("metric_without_the_norm",
     "return np.abs(np.asarray(W, dtype=F64)) * np.asarray(xnorm, dtype=F64)[None, :]",
     "return np.abs(np.asarray(W, dtype=F64)) + 0.0 * np.asarray(xnorm, dtype=F64)[None, :]"),
    ("psi_takes_the_largest", "M[order[: int(r)]] = 1", "M[order[::-1][: int(r)]] = 1"),
    ("nm_takes_the_largest", "M[i, g0 + order[:k]] = 1", "M[i, g0 + order[::-1][:k]] = 1"),
    ("update_with_the_wrong_sign", "return -(lam @ R), lam", "return (lam @ R), lam"),
    ("rows_of_the_inverse_transposed_away", "R = Hinv[q, :]\n    Rhat = R[:, q]\n    u = w[q]\n    lam",
     "R = Hinv[q, :] * (1.0 + 0.01 * np.arange(Hinv.shape[0]))[None, :]\n    Rhat = R[:, q]\n    u = w[q]\n    lam"),
    ("full_instead_of_residual_inverse", "Hinv = np.linalg.inv(Hd[j1:, j1:])",
     "Hinv = np.linalg.inv(Hd)[j1:, j1:]"),
    ("budget_not_decremented", 'state["r"] -= int(Mb.sum())', 'state["r"] -= 0'),
    ("removed_weights_not_forced_to_zero", "Wc[i, j1 + q] = 0.0", "Wc[i, j1 + q] += 1e-9"),
    ("row_losses_without_the_half", 'return 0.5 * np.einsum("ij,jk,ik->i"', 'return 1.0 * np.einsum("ij,jk,ik->i"'),
    ("outliers_are_the_smallest_losses", 'sigma = np.argsort(h, kind="stable")\n    return sigma, n_out',
     'sigma = np.argsort(-h, kind="stable")\n    return sigma, n_out'),
    ("column_losses_without_the_norm",
     "return np.sum(W_rows ** 2, axis=0) * np.asarray(xnorm, dtype=F64) ** 2",
     "return np.sum(W_rows ** 2, axis=0) + 0.0 * np.asarray(xnorm, dtype=F64)"),
    ("structured_count_rounded_down", "return int(math.ceil(float(p) * b / (1.0 - float(alpha)) - 1e-12))",
     "return int(math.floor(float(p) * b / (1.0 - float(alpha))))"),
    ("structured_takes_the_largest_columns", 'sigma_c = np.argsort(v, kind="stable")',
     'sigma_c = np.argsort(-v, kind="stable")'),
    ("structured_update_with_the_wrong_sign", "Wp[:n_rows] = Wp[:n_rows] - lam @ Hinv[:s, :]",
     "Wp[:n_rows] = Wp[:n_rows] + lam @ Hinv[:s, :]"),
    ("structured_outlier_rows_updated", "Wp[:n_rows] = Wp[:n_rows] - lam @ Hinv[:s, :]",
     "Wp[:n_rows] = Wp[:n_rows] - lam @ Hinv[:s, :]\n        Wp[n_rows:, :s] = 0.0"),
]


def _pin_calls():
    """Every pin with its arguments (parametrised ones once per parameter set)."""
    calls = []
    for name, fn in sorted(vars(pins).items()):
        if not name.startswith("test_") or not callable(fn):
            continue
        marks = [m for m in getattr(fn, "pytestmark", []) if m.name == "parametrize"]
        if not marks:
            calls.append((name, fn, {}))
            continue
        names, values = marks[0].args[0], marks[0].args[1]
        names = [s.strip() for s in names.split(",")]
        for v in values:
            v = v if isinstance(v, (tuple, list)) and len(names) > 1 else (v,)
            calls.append((name, fn, dict(zip(names, v))))
    return calls


def _failing_pins(module):
    failed = []
    saved = pins.O
    pins.O = module
    try:
        for name, fn, kw in _pin_calls():
            try:
                fn(**kw)
            except Exception:  # an assertion, or an exception the mistake provokes
                failed.append(name)
    finally:
        pins.O = saved
    return failed


def test_the_unmodified_oracle_passes_through_this_harness():
    assert _failing_pins(O) == []
    assert len(_pin_calls()) >= 30


@pytest.mark.parametrize("name,old,new", [m for m in MUTANTS if m[1] is not None],
                         ids=[m[0] for m in MUTANTS if m[1] is not None])
def test_pins_notice_a_planted_mistake(name, old, new):
    assert SRC.count(old) >= 1, "the oracle no longer contains the text this case rewrites"
    mod = types.ModuleType("oracle_mutant_" + name)
    mod.__file__ = O.__file__
    exec(compile(SRC.replace(old, new, 1), O.__file__, "exec"), mod.__dict__)
    failed = _failing_pins(mod)
    assert failed, "no pin noticed: " + name
