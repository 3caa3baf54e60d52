"""Pins of the SDCA oracle (l2-regularised multiclass logistic regression, Section 2.1 "Stochastic DCA"): what the
mathematics fixes, checked with routines the oracle does not use (scipy's minimisers and root finder)."""
import numpy as np
import pytest
from scipy.optimize import brentq, minimize

from oracle import sdca_oracle as D


def _problem(N=24, J=4, Dm=5, seed=0):
    rng = np.random.default_rng(seed)
    A = rng.normal(size=(N, Dm))
    y = rng.integers(0, J, size=N)
    return A, y


def _random_simplex(rng, n, J):
    Q = rng.exponential(size=(n, J))
    return Q / Q.sum(axis=1, keepdims=True)


def test_coordinate_minimiser_is_the_constrained_minimum():
    rng = np.random.default_rng(1)
    for kappa in (0.0, 0.03, 0.7, 5.0):
        z = rng.normal(size=4) * 2
        q_old = _random_simplex(rng, 1, 4)[0]
        q = D.coordinate_minimiser(z, q_old, kappa)
        assert abs(q.sum() - 1) < 1e-12 and (q > 0).all()

        def phi(p):
            return float(np.sum(p * np.log(p)) - p @ (z + kappa * q_old) + 0.5 * kappa * p @ p)
        # scipy's BFGS over the simplex written as q = softmax(theta) (an unconstrained problem), from two starts
        def soft(th):
            e = np.exp(th - th.max())
            return e / e.sum()
        best = min((minimize(lambda th: phi(soft(th)), x0, method="BFGS", options={"gtol": 1e-12, "maxiter": 2000})
                    for x0 in (np.zeros(4), np.log(q_old))), key=lambda r: r.fun)
        assert phi(q) <= best.fun + 1e-10
        np.testing.assert_allclose(q, soft(best.x), atol=2e-5)
        # stationarity: log q_j + kappa q_j - t_j is the same constant for every j
        r = np.log(q) + kappa * q - (z + kappa * q_old)
        assert np.ptp(r) < 1e-10


def test_two_classes_reduce_to_one_scalar_equation():
    """J = 2: subtracting the two stationarity conditions leaves logit(q) + kappa (2q - 1) = t_1 - t_2."""
    rng = np.random.default_rng(2)
    for _ in range(5):
        z, q_old, kappa = rng.normal(size=2) * 3, _random_simplex(rng, 1, 2)[0], float(rng.uniform(0.01, 3))
        t = z + kappa * q_old
        root = brentq(lambda q: np.log(q / (1 - q)) + kappa * (2 * q - 1) - (t[0] - t[1]), 1e-15, 1 - 1e-15, xtol=1e-15)
        q = D.coordinate_minimiser(z, q_old, kappa)
        assert abs(q[0] - root) < 1e-12


def test_without_the_quadratic_term_the_minimiser_is_the_softmax():
    z = np.array([0.3, -1.0, 2.0])
    e = np.exp(z - z.max())
    np.testing.assert_allclose(D.coordinate_minimiser(z, np.array([1.0, 0, 0]), 0.0), e / e.sum(), atol=1e-14)
    np.testing.assert_allclose(D.coordinate_minimiser(z, np.array([1.0, 0, 0]), 1e-9), e / e.sum(), atol=1e-8)


def test_weak_duality_for_any_feasible_dual_state():
    A, y = _problem()
    rng = np.random.default_rng(3)
    for lam in (0.1, 1.0):
        for _ in range(5):
            Q = _random_simplex(rng, len(y), 4)
            W = D.w_from_dual(Q, A, y, lam)
            assert D.l2mlr_primal(W, A, y, lam) + D.l2mlr_dual(Q, A, y, lam) >= -1e-12
    Q0 = D.initial_dual(y, 4)
    assert np.all(D.w_from_dual(Q0, A, y, 0.1) == 0) and D.l2mlr_dual(Q0, A, y, 0.1) == 0.0
    assert abs(D.l2mlr_primal(np.zeros((4, 5)), A, y, 0.1) - np.log(4)) < 1e-12          # gap at the start: log J


def test_dual_objective_never_increases_and_W_tracks_the_dual_state():
    A, y = _problem(N=24)
    lam, N = 0.1, 24
    rng = np.random.default_rng(4)
    for K, gamma, workers in ((1, 1.0, 1), (6, 1.0 / 6, 3), (8, 1.0 / 8, 2)):
        Q = D.initial_dual(y, 4)
        W = np.zeros((4, 5))
        prev = D.l2mlr_dual(Q, A, y, lam)
        for step in range(30):
            ids = rng.choice(N, size=K, replace=False)
            W, Q, U, V = D.sdca_step(W, A[ids], y[ids], ids, Q, lam, gamma, workers)
            cur = D.l2mlr_dual(Q, A, y, lam)
            assert cur <= prev + 1e-13, (K, step)
            prev = cur
            assert np.allclose(Q.sum(axis=1), 1) and (Q >= 0).all()
            # the factors sum to zero over the classes (both q's are on the simplex)
            assert np.abs(U.sum(axis=1)).max() < 1e-12
        np.testing.assert_allclose(W, D.w_from_dual(Q, A, y, lam), atol=1e-13)        # W = grad h*(Z) of the state


def test_single_sample_step_is_the_exact_coordinate_minimum_of_the_dual():
    """After the step on sample i, no other feasible value of q_i gives a smaller (D)."""
    A, y = _problem(N=10, J=3, Dm=4, seed=5)
    lam = 0.2
    rng = np.random.default_rng(6)
    Q = _random_simplex(rng, 10, 3)
    W = D.w_from_dual(Q, A, y, lam)
    i = 7
    _, Q1, _, _ = D.sdca_step(W, A[[i]], y[[i]], [i], Q, lam, 1.0)
    best = D.l2mlr_dual(Q1, A, y, lam)
    for _ in range(300):
        Qt = Q1.copy()
        Qt[i] = _random_simplex(rng, 1, 3)[0] if rng.random() < 0.5 else np.abs(Q1[i] + 1e-3 * rng.normal(size=3))
        Qt[i] /= Qt[i].sum()
        assert D.l2mlr_dual(Qt, A, y, lam) >= best - 1e-13


def test_sweeps_close_the_gap_and_reach_the_primal_optimum():
    A, y = _problem(N=24)
    lam, N, J = 0.1, 24, 4
    Q, W = D.initial_dual(y, J), np.zeros((J, 5))
    gaps = []
    for sweep in range(60):
        for i in range(N):
            W, Q, _, _ = D.sdca_step(W, A[[i]], y[[i]], [i], Q, lam, 1.0)
        gaps.append(D.l2mlr_primal(W, A, y, lam) + D.l2mlr_dual(Q, A, y, lam))
    assert gaps[0] < np.log(J) and gaps[-1] < 1e-9 and all(g >= -1e-12 for g in gaps)
    assert all(b <= a + 1e-12 for a, b in zip(gaps, gaps[1:]))
    opt = minimize(lambda w: D.l2mlr_primal(w.reshape(J, 5), A, y, lam), np.zeros(J * 5), method="L-BFGS-B",
                   options={"ftol": 1e-16, "gtol": 1e-10, "maxiter": 5000})
    np.testing.assert_allclose(W, opt.x.reshape(J, 5), atol=2e-5)
    # at the optimum every dual vector is the prediction: q_i = softmax(W a_i), and the factors vanish
    Z = A @ W.T
    Pm = np.exp(Z - Z.max(axis=1, keepdims=True))
    Pm /= Pm.sum(axis=1, keepdims=True)
    np.testing.assert_allclose(Q, Pm, atol=1e-5)
    U, _ = D.sdca_factors(W, A, y, Q, lam, N)
    assert np.abs(U).max() < 1e-5


def test_hand_worked_case_two_classes_one_sample():
    """N = 1, J = 2, a = (1), y = 0, lam = 1, from W = 0 (q_old = e_0): kappa = 1, t = (1, 0); the conditions
    log q + q = 1 - nu, log(1 - q) + (1 - q) = -nu give logit(q) + 2q - 1 = 1, whose root is q = 0.70349...
    (checked by hand: logit(0.7035) = 0.8639, 2 * 0.7035 - 1 = 0.4070, sum 1.2709 ... see the closed form below)."""
    q = D.coordinate_minimiser(np.zeros(2), np.array([1.0, 0.0]), 1.0)
    # independent statement of the root: logit(q) + 2 q = 2  ->  solve by brentq
    root = brentq(lambda p: np.log(p / (1 - p)) + 2 * p - 2, 1e-12, 1 - 1e-12, xtol=1e-15)
    assert abs(q[0] - root) < 1e-12 and 0.5 < q[0] < 1.0
    W1, Q1, U, V = D.sdca_step(np.zeros((2, 1)), np.array([[1.0]]), np.array([0]), [0], D.initial_dual([0], 2), 1.0, 1.0)
    np.testing.assert_allclose(U, [[root - 1.0, 1.0 - root]], atol=1e-12)          # du = q_new - q_old
    np.testing.assert_allclose(W1, [[1.0 - root], [root - 1.0]], atol=1e-12)        # W = (e_0 - q) a^T / (lam N)
