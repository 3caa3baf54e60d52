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
             T.test_comm_values_count_what_is_moved, T.test_sampled_mlr_helpers_match_the_plain_step,
             T.test_entrywise_prox_operators_solve_their_defining_problem]
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
                                    "prox_unit_columns", "gather", "ista_codes", "lipschitz_power_iteration",
                                    "prox_l1", "prox_l2sq")}

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
    "prox l1: threshold halved": ("prox_l1", lambda W, t: ORIG["prox_l1"](W, 0.5 * t)),
    "prox l2: divided by 1 + 2t": ("prox_l2sq", lambda W, t: ORIG["prox_l2sq"](W, 2 * t)),
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


# ----------------------------------------------------------------------------------------------------------
# The same for the SDCA oracle: mistakes planted in oracle/sdca_oracle.py must fail a pin of test_sdca_pins.py
# ----------------------------------------------------------------------------------------------------------
from oracle import sdca_oracle as D   # noqa: E402
import test_sdca_pins as TS           # noqa: E402

SDCA_PINS = [TS.test_coordinate_minimiser_is_the_constrained_minimum, TS.test_two_classes_reduce_to_one_scalar_equation,
             TS.test_without_the_quadratic_term_the_minimiser_is_the_softmax,
             TS.test_weak_duality_for_any_feasible_dual_state,
             TS.test_dual_objective_never_increases_and_W_tracks_the_dual_state,
             TS.test_single_sample_step_is_the_exact_coordinate_minimum_of_the_dual,
             TS.test_sweeps_close_the_gap_and_reach_the_primal_optimum,
             TS.test_hand_worked_case_two_classes_one_sample]
DORIG = {n: getattr(D, n) for n in ("coordinate_minimiser", "sdca_factors", "sdca_step", "w_from_dual", "l2mlr_dual")}


def _sdca_caught():
    for pin in SDCA_PINS:
        try:
            pin()
        except Exception:
            return True
    return False


def _factors_sign(W, X, y, Q_rows, lam, N):
    U, V = DORIG["sdca_factors"](W, X, y, Q_rows, lam, N)
    return -U, V


def _factors_kappa_without_norm(W, X, y, Q_rows, lam, N):
    X = np.asarray(X, dtype=np.float64)
    Z = X @ np.asarray(W, dtype=np.float64).T
    U = np.stack([DORIG["coordinate_minimiser"](Z[i], Q_rows[i], 1.0 / (lam * N)) - Q_rows[i] for i in range(len(X))])
    return U, X.copy()


def _step_without_one_over_N(W, X, y, ids, Q, lam, gamma, workers=1):
    W1, Q1, U, V = DORIG["sdca_step"](W, X, y, ids, Q, lam, gamma, workers)
    return np.asarray(W, dtype=np.float64) - (gamma / lam) * (U.T @ V), Q1, U, V


def _step_dual_not_damped(W, X, y, ids, Q, lam, gamma, workers=1):
    W1, Q1, U, V = DORIG["sdca_step"](W, X, y, ids, Q, lam, gamma, workers)
    Q2 = np.asarray(Q, dtype=np.float64).copy()
    Q2[np.asarray(ids)] += U                                  # gamma forgotten on the dual side only
    return W1, Q2, U, V


SDCA_MUTATIONS = {
    "sdca: du with the wrong sign": ("sdca_factors", _factors_sign),
    "sdca: kappa without ||a||^2": ("sdca_factors", _factors_kappa_without_norm),
    "sdca: quadratic term ignored (plain softmax)": ("coordinate_minimiser", lambda z, q_old, kappa, iters=200: DORIG["coordinate_minimiser"](z, q_old, 0.0)),
    "sdca: q_old dropped from the right-hand side": ("coordinate_minimiser", lambda z, q_old, kappa, iters=200: DORIG["coordinate_minimiser"](z, np.zeros_like(q_old), kappa)),
    "sdca: Z updated without 1/N": ("sdca_step", _step_without_one_over_N),
    "sdca: dual state moved by the undamped change": ("sdca_step", _step_dual_not_damped),
    "sdca: W = Z (1/lam dropped)": ("w_from_dual", lambda Q, A, y, lam: lam * DORIG["w_from_dual"](Q, A, y, lam)),
    "sdca: conjugate with the wrong sign": ("l2mlr_dual", lambda Q, A, y, lam: DORIG["l2mlr_dual"](Q, A, y, lam) - 2 * float(np.where(np.asarray(Q) > 0, Q * np.log(np.where(np.asarray(Q) > 0, Q, 1.0)), 0.0).sum()) / len(y)),
}


def test_unmutated_sdca_oracle_passes_every_pin():
    assert not _sdca_caught()


@pytest.mark.parametrize("name", sorted(SDCA_MUTATIONS))
def test_a_planted_sdca_mistake_is_caught_by_some_pin(name, monkeypatch):
    attr, fn = SDCA_MUTATIONS[name]
    monkeypatch.setattr(D, attr, fn)
    assert _sdca_caught(), f"no pin noticed: {name}"
