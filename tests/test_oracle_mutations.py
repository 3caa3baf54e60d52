"""The pins must be able to fail: a plausible mistake planted in the oracle (a dropped term, a wrong sign or
constant, a flipped branch, a swapped order) has to be caught by at least one pin of tests/test_oracle_pins.py.
Every mistake is planted in the oracle, on the CPU, and removed again."""
import numpy as np
import pytest

from oracle import sfb_oracle as O
import test_oracle_pins as T


def _pins():
    pins = [lambda c=c: T.test_hand_worked_cases(c) for c in T._golden()]
    pins += [T.test_mlr_factors_match_finite_differences, T.test_dml_factors_match_finite_differences,
             T.test_sc_factors_match_finite_differences, T.test_update_rank_at_most_K,
             T.test_gather_is_worker_major_and_split_invariant, T.test_mlr_zero_init_closed_form,
             T.test_mlr_invariants, T.test_dml_three_matmul_closed_form, T.test_sc_closed_form_and_ista_properties,
             T.test_prox_properties, T.test_power_iteration_matches_spectral_norm,
             T.test_comm_values_count_what_is_moved, T.test_sampled_mlr_helpers_match_the_plain_step]
    pins += [lambda m=m: T.test_reconstruction_equals_dense_gradient_and_dense_sync(m) for m in (O.MLR, O.DML, O.SC)]
    return pins


def _caught():
    for pin in _pins():
        try:
            pin()
        except Exception:          # an assertion, or a shape error from a transposed operand: both are "caught"
            return True
    return False


def _mlr_without_onehot(W, X, y):
    U, V = ORIG["mlr_factors"](W, X, y)
    U[np.arange(U.shape[0]), np.asarray(y, dtype=np.int64)] += 1.0
    return U, V


def _dml_factor_one(W, X, Y, similar, margin=1.0):
    U, V = ORIG["dml_factors"](W, X, Y, similar, margin)
    return 0.5 * U, V


def _dml_hinge_flipped(W, X, Y, similar, margin=1.0):
    W = np.asarray(W, dtype=np.float64)
    V = np.asarray(X, dtype=np.float64) - np.asarray(Y, dtype=np.float64)
    Z = V @ W.T
    q = (Z * Z).sum(axis=1)
    s = np.where(np.asarray(similar) != 0, 1.0, np.where(q > margin, -1.0, 0.0))
    return 2.0 * s[:, None] * Z, V


def _dml_pair_sum(W, X, Y, similar, margin=1.0):
    return ORIG["dml_factors"](W, X, -np.asarray(Y, dtype=np.float64), similar, margin)


ORIG = {n: getattr(O, n) for n in ("mlr_factors", "dml_factors", "soft_threshold", "rank_k_update",
                                    "prox_unit_columns", "gather", "ista_codes", "lipschitz_power_iteration")}

MUTATIONS = {
    "mlr: onehot(y) not subtracted": ("mlr_factors", _mlr_without_onehot),
    "dml: factor 2 dropped": ("dml_factors", _dml_factor_one),
    "dml: hinge branch flipped": ("dml_factors", _dml_hinge_flipped),
    "dml: x + y instead of x - y": ("dml_factors", _dml_pair_sum),
    "sc: no shrinkage": ("soft_threshold", lambda w, t: w),
    "sc: threshold twice too large": ("soft_threshold", lambda w, t: ORIG["soft_threshold"](w, 2 * t)),
    "update: sign": ("rank_k_update", lambda W, U, V, eta: np.asarray(W, dtype=np.float64) + eta * (np.asarray(U).T @ np.asarray(V))),
    "update: eta squared": ("rank_k_update", lambda W, U, V, eta: ORIG["rank_k_update"](W, U, V, eta * eta)),
    "update: U and V swapped": ("rank_k_update", lambda W, U, V, eta: ORIG["rank_k_update"](W, V, U, eta)),
    "prox: every column rescaled": ("prox_unit_columns", lambda W: np.asarray(W, dtype=np.float64) / np.sqrt((np.asarray(W, dtype=np.float64) ** 2).sum(axis=0))),
    "gather: workers in reverse order": ("gather", lambda fs: ORIG["gather"](list(reversed(fs)))),
    "ista: one iteration too few": ("ista_codes", lambda W, X, lam, L, iters: ORIG["ista_codes"](W, X, lam, L, max(iters - 1, 0))),
    "power iteration: norm, not its square": ("lipschitz_power_iteration", lambda W, iters=50: float(np.sqrt(ORIG["lipschitz_power_iteration"](W, iters)))),
}


def test_unmutated_oracle_passes_every_pin():
    assert not _caught()


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_a_planted_mistake_is_caught_by_some_pin(name, monkeypatch):
    attr, fn = MUTATIONS[name]
    monkeypatch.setattr(O, attr, fn)
    assert _caught(), f"no pin noticed: {name}"
