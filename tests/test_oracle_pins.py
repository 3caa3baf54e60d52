"""Pins for the fp64 oracle: what the paper and the mathematics fix, independent of the oracle's own code.

Each test names the passage of the paper it rests on.  None of these needs a GPU.
"""
import ast
import math
import os

import numpy as np
import pytest

from oracle import sfb_oracle as O

HERE = os.path.dirname(os.path.abspath(__file__))
rng = np.random.default_rng(1234)


def _golden():
    cases = []
    with open(os.path.join(HERE, "golden", "hand_worked_cases.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            cases.append(ast.literal_eval(line))
    return cases


def _arr(v):
    def conv(e):
        if isinstance(e, list):
            return [conv(x) for x in e]
        return math.log(2.0) if e == "ln2" else e
    return np.array(conv(v), dtype=np.float64)


@pytest.mark.parametrize("case", _golden(), ids=lambda c: c["case"])
def test_hand_worked_cases(case):
    """Hand-derived values (tests/golden/hand_worked_cases.txt), Sections 2, 2.1, 3 and Figure 3."""
    kind = case["case"]
    if kind == "mlr":
        U, V = O.mlr_factors(_arr(case["W"]), _arr(case["x"]), np.array(case["y"]))
        np.testing.assert_allclose(U, _arr(case["u"]), atol=1e-15)
        np.testing.assert_allclose(V, _arr(case["v"]), atol=0)
    elif kind == "dml":
        U, V = O.dml_factors(_arr(case["W"]), _arr(case["x"]), _arr(case["y"]), np.array(case["similar"]), 1.0)
        np.testing.assert_allclose(U, _arr(case["u"]), atol=1e-15)
        np.testing.assert_allclose(V, _arr(case["v"]), atol=0)
    elif kind == "sc":
        U, A = O.sc_factors(_arr(case["W"]), _arr(case["x"]), case["lam"], case["L"], case["iters"])
        np.testing.assert_allclose(A, _arr(case["a"]), atol=1e-14)
        np.testing.assert_allclose(U, _arr(case["u"]), atol=1e-14)
    elif kind == "prox":
        np.testing.assert_allclose(O.prox_unit_columns(_arr(case["W"])), _arr(case["out"]), atol=1e-15)
    elif kind == "update":
        out = O.rank_k_update(_arr(case["W"]), _arr(case["U"]), _arr(case["V"]), case["eta"])
        np.testing.assert_allclose(out, _arr(case["out"]), atol=1e-15)
    else:
        raise AssertionError(kind)


# ----------------------------------------------------------------------------------------------------------
# u = d f / d (W a), v = a (Section 2.1): central finite differences of each loss w.r.t. every entry of W
# ----------------------------------------------------------------------------------------------------------
def _fd_grad(loss, W, h=1e-6):
    G = np.zeros_like(W)
    for j in range(W.shape[0]):
        for d in range(W.shape[1]):
            Wp, Wm = W.copy(), W.copy()
            Wp[j, d] += h
            Wm[j, d] -= h
            G[j, d] = (loss(Wp).sum() - loss(Wm).sum()) / (2 * h)
    return G


def test_mlr_factors_match_finite_differences():
    J, D, K = 5, 7, 6
    W = rng.normal(size=(J, D))
    X = rng.normal(size=(K, D))
    y = rng.integers(0, J, size=K)
    U, V = O.mlr_factors(W, X, y)
    G = _fd_grad(lambda Wx: O.mlr_loss(Wx, X, y), W)
    np.testing.assert_allclose(U.T @ V, G, rtol=1e-6, atol=1e-8)


def test_dml_factors_match_finite_differences():
    k, D, K = 4, 6, 8
    W = 0.25 * rng.normal(size=(k, D))
    X = rng.normal(size=(K, D))
    Y = rng.normal(size=(K, D))
    sim = np.array([1, 0, 1, 0, 0, 1, 0, 0])
    Y[1] = X[1] + 0.3 * Y[1]                     # two close dissimilar pairs: active hinge
    Y[4] = X[4] + 0.3 * Y[4]
    U, V = O.dml_factors(W, X, Y, sim, 1.0)
    q = (((X - Y) @ W.T) ** 2).sum(axis=1)
    # the batch must exercise both the active and the inactive hinge branch, away from the kink
    dis = sim == 0
    assert (q[dis] < 0.9).any() and (q[dis] > 1.1).any()
    G = _fd_grad(lambda Wx: O.dml_loss(Wx, X, Y, sim, 1.0), W)
    np.testing.assert_allclose(U.T @ V, G, rtol=1e-6, atol=1e-7)


def test_sc_factors_match_finite_differences():
    D, A, K = 6, 5, 4
    W = rng.normal(size=(D, A))
    X = rng.normal(size=(K, D))
    L = np.linalg.norm(W, 2) ** 2
    U, V = O.sc_factors(W, X, 0.1, L, 20)
    G = _fd_grad(lambda Wx: O.sc_loss(Wx, V, X), W)
    np.testing.assert_allclose(U.T @ V, G, rtol=1e-6, atol=1e-7)


# ----------------------------------------------------------------------------------------------------------
# "the update can be exactly constructed from the SFs" (Section 1), Figure 1: sum u v^T equals the
# minibatch gradient computed without factors; SFB and full-matrix sync make the same progress (Experiments)
# ----------------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("model", [O.MLR, O.DML, O.SC])
def test_reconstruction_equals_dense_gradient_and_dense_sync(model):
    P, B = 3, 4
    K = P * B
    if model == O.MLR:
        W = rng.normal(size=(6, 9)); X = rng.normal(size=(K, 9)); Y = None
        lab = rng.integers(0, 6, size=K); kw = {}
    elif model == O.DML:
        W = 0.2 * rng.normal(size=(5, 8)); X = rng.normal(size=(K, 8)); Y = rng.normal(size=(K, 8))
        lab = rng.integers(0, 2, size=K); kw = {}
    else:
        W = rng.normal(size=(9, 6)); X = rng.normal(size=(K, 9)); Y = None; lab = None
        kw = dict(lam=0.1, L=np.linalg.norm(W, 2) ** 2, iters=20)
    eta = 0.05
    Wn, U, V = O.sfb_step(model, W, X, Y, lab, workers=P, eta=eta, return_factors=True,
                          prox=(model == O.SC), **kw)
    G = O.dense_gradient(model, W, X, Y, lab, 1.0, codes=V if model == O.SC else None)
    np.testing.assert_allclose(U.T @ V, G, rtol=1e-12, atol=1e-13)
    Wd = O.dense_sync_step(model, W, X, Y, lab, workers=P, eta=eta, codes=V if model == O.SC else None,
                           prox=(model == O.SC))
    np.testing.assert_allclose(Wn, Wd, rtol=1e-12, atol=1e-13)


def test_update_rank_at_most_K():
    """A minibatch of K pairs gives an update of rank <= K (Section 2.1, low-rank extensions)."""
    J, D, K = 32, 48, 5
    W = rng.normal(size=(J, D)); X = rng.normal(size=(K, D)); y = rng.integers(0, J, size=K)
    U, V = O.mlr_factors(W, X, y)
    s = np.linalg.svd(U.T @ V, compute_uv=False)
    assert s[K - 1] > 1e-6 * s[0]
    assert s[K] <= 1e-12 * s[0]


def test_gather_is_worker_major_and_split_invariant():
    """Section 3: each worker's K pairs are broadcast whole; BSP => the result does not depend on how the
    same samples are split over workers."""
    J, D, K = 7, 5, 24
    W = rng.normal(size=(J, D)); X = rng.normal(size=(K, D)); y = rng.integers(0, J, size=K)
    W1, U1, V1 = O.sfb_step(O.MLR, W, X, None, y, workers=1, eta=0.1, return_factors=True)
    W4, U4, V4 = O.sfb_step(O.MLR, W, X, None, y, workers=4, eta=0.1, return_factors=True)
    np.testing.assert_array_equal(V4, X)           # row i = p*B + b keeps the sample order
    np.testing.assert_allclose(U4, U1, atol=1e-15)
    np.testing.assert_allclose(W4, W1, atol=1e-14)
    perm = rng.permutation(K)
    np.testing.assert_allclose(O.rank_k_update(W, U1[perm], V1[perm], 0.1), W1, atol=1e-13)


# ----------------------------------------------------------------------------------------------------------
# MLR closed form and invariants
# ----------------------------------------------------------------------------------------------------------
def test_mlr_zero_init_closed_form():
    """W = 0 => p = 1/J for every class: Delta W = (1/J) 1 (sum_i x_i)^T - sum_i e_{y_i} x_i^T."""
    J, D, K = 8, 5, 16
    X = rng.normal(size=(K, D)); y = rng.integers(0, J, size=K)
    Wn = O.sfb_step(O.MLR, np.zeros((J, D)), X, None, y, workers=4, eta=0.01)
    dW = np.tile(X.sum(axis=0) / J, (J, 1))
    for i in range(K):
        dW[y[i]] -= X[i]
    np.testing.assert_allclose(Wn, -0.01 * dW, atol=1e-15)


def test_mlr_invariants():
    J, D, K = 11, 6, 9
    W = rng.normal(size=(J, D)); X = rng.normal(size=(K, D)); y = rng.integers(0, J, size=K)
    U, V = O.mlr_factors(W, X, y)
    np.testing.assert_allclose(U.sum(axis=1), 0.0, atol=1e-14)
    lab = U[np.arange(K), y]
    assert ((lab > -1) & (lab < 0)).all()
    U2 = U.copy(); U2[np.arange(K), y] += 1.0
    assert ((U2 > 0) & (U2 < 1)).all()
    Wn = O.rank_k_update(W, U, V, 0.3)
    np.testing.assert_allclose(Wn.sum(axis=0), W.sum(axis=0), atol=1e-13)   # 1^T Delta W = 0
    # adding one vector to every row of W shifts all logits of a sample alike: softmax unchanged
    Wc = W + np.outer(np.ones(J), rng.normal(size=D))                      # same vector added to every row
    Uc, _ = O.mlr_factors(Wc, X, y)
    np.testing.assert_allclose(Uc, U, atol=1e-12)


# ----------------------------------------------------------------------------------------------------------
# DML and SC closed forms through library matmuls
# ----------------------------------------------------------------------------------------------------------
def test_dml_three_matmul_closed_form():
    k, D, K = 6, 10, 12
    W = 0.2 * rng.normal(size=(k, D)); X = rng.normal(size=(K, D)); Y = rng.normal(size=(K, D))
    sim = rng.integers(0, 2, size=K)
    V = X - Y
    q = np.einsum("kd,jd,je,ke->k", V, W, W, V)
    s = np.where(sim == 1, 1.0, np.where(q < 1.0, -1.0, 0.0))
    dW = 2.0 * W @ V.T @ np.diag(s) @ V
    Wn = O.sfb_step(O.DML, W, X, Y, sim, workers=3, eta=1e-2)
    np.testing.assert_allclose(Wn, W - 1e-2 * dW, rtol=1e-12, atol=1e-14)


def test_sc_closed_form_and_ista_properties():
    D, A, K = 12, 8, 6
    W = rng.normal(size=(D, A)); W /= np.linalg.norm(W, axis=0)
    X = rng.normal(size=(K, D))
    L = np.linalg.norm(W, 2) ** 2
    lam = 0.1
    # the objective never increases for step 1/L (ISTA, the proximal-gradient method the paper builds on)
    prev = O.sc_objective(W, np.zeros((K, A)), X, lam)
    for t in range(1, 25):
        cur = O.sc_objective(W, O.ista_codes(W, X, lam, L, t), X, lam)
        assert (cur <= prev + 1e-12).all()
        prev = cur
    # many iterations reach the lasso optimum: 0 in the subdifferential
    Aopt = O.ista_codes(W, X, lam, L, 5000)
    G = (Aopt @ W.T - X) @ W
    on = Aopt != 0
    np.testing.assert_allclose(G[on], -lam * np.sign(Aopt[on]), atol=1e-8)
    assert (np.abs(G[~on]) <= lam + 1e-8).all()
    # a = 0 is a fixed point when lam >= ||W^T x||_inf
    big = np.abs(X @ W).max() + 1e-9
    assert (O.ista_codes(W, X, big, L, 7) == 0).all()
    # orthonormal dictionary, L = 1: one iteration gives soft(W^T x, lam) and stays there
    Q, _ = np.linalg.qr(rng.normal(size=(D, A)))
    expect = np.sign(X @ Q) * np.maximum(np.abs(X @ Q) - lam, 0)
    np.testing.assert_allclose(O.ista_codes(Q, X, lam, 1.0, 1), expect, atol=1e-14)
    np.testing.assert_allclose(O.ista_codes(Q, X, lam, 1.0, 9), expect, atol=1e-13)
    # step closed form: Delta W = (W A^T - X^T) A
    Wn, U, V = O.sfb_step(O.SC, W, X, workers=2, eta=1e-3, lam=lam, L=L, iters=20, return_factors=True)
    np.testing.assert_allclose(Wn, W - 1e-3 * (W @ V.T - X.T) @ V, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(V, O.ista_codes(W, X, lam, L, 20), atol=0)


def test_prox_properties():
    """Figure 3: only columns of norm > 1 are rescaled, to norm exactly 1."""
    W = rng.normal(size=(10, 7))
    W[:, 0] *= 0.01; W[:, 3] *= 0.05
    Pw = O.prox_unit_columns(W)
    n0 = np.linalg.norm(W, axis=0)
    small = n0 <= 1
    assert small.any() and (~small).any()
    assert (np.linalg.norm(Pw, axis=0) <= 1 + 1e-15).all()
    np.testing.assert_array_equal(Pw[:, small], W[:, small])
    np.testing.assert_allclose(np.linalg.norm(Pw[:, ~small], axis=0), 1.0, atol=1e-15)
    np.testing.assert_allclose(O.prox_unit_columns(Pw), Pw, atol=1e-15)
    # it is the Euclidean projection: no feasible point is closer
    for _ in range(20):
        C = rng.normal(size=W.shape); C /= np.maximum(1.0, np.linalg.norm(C, axis=0))
        assert np.linalg.norm(W - Pw) <= np.linalg.norm(W - C) + 1e-12


def test_power_iteration_matches_spectral_norm():
    W = rng.normal(size=(40, 25))
    assert abs(O.lipschitz_power_iteration(W, 400) - np.linalg.norm(W, 2) ** 2) < 1e-8 * np.linalg.norm(W, 2) ** 2
    # 50 iterations never overshoot (Rayleigh quotient) and are close
    L50 = O.lipschitz_power_iteration(W, 50)
    assert L50 <= np.linalg.norm(W, 2) ** 2 * (1 + 1e-12)
    assert L50 >= 0.9 * np.linalg.norm(W, 2) ** 2


def test_comm_values_count_what_is_moved():
    """Section 5 cost table: count the entries of the arrays actually exchanged."""
    J, D, P, B = 7, 5, 3, 4
    W = rng.normal(size=(J, D)); X = rng.normal(size=(P * B, D)); y = rng.integers(0, J, size=P * B)
    per_worker = [O.mlr_factors(W, X[p * B:(p + 1) * B], y[p * B:(p + 1) * B]) for p in range(P)]
    one = sum(u.size + v.size for u, v in per_worker)
    p2p = sum((u.size + v.size) * (P - 1) for u, v in per_worker)
    fms = sum(W.size for _ in range(P))
    assert O.comm_values(J, D, P, B) == (one, p2p, fms)


def test_sampled_mlr_helpers_match_the_plain_step():
    J, D, K = 37, 9, 10
    W = rng.normal(size=(J, D)).astype(np.float32); X = rng.normal(size=(K, D)).astype(np.float32)
    y = rng.integers(0, J, size=K)
    Z = X.astype(np.float64) @ W.astype(np.float64).T
    lse_ref = np.log(np.exp(Z).sum(axis=1))
    lse = O.mlr_log_partition(W, X, block_rows=8)
    np.testing.assert_allclose(lse, lse_ref, rtol=1e-14)
    Wn = O.sfb_step(O.MLR, W, X, None, y, workers=2, eta=0.05)
    rows = np.array([0, 5, 36, int(y[0])])
    np.testing.assert_allclose(O.mlr_updated_rows(W[rows], rows, X, y, lse, 0.05), Wn[rows], atol=1e-14)


def test_entrywise_prox_operators_solve_their_defining_problem():
    """prox_{t h}(w) = argmin_v 1/2 (v - w)^2 + t h(v) (Section 2.1, proximal SGD), entry by entry: checked against
    scipy's bounded scalar minimiser, which the oracle does not use; plus what the definition implies."""
    from scipy.optimize import minimize_scalar
    rng = np.random.default_rng(12)
    w = np.concatenate([rng.normal(size=12), [0.0, 0.3, -0.3, 0.3000001, 1e-9]])
    for t in (0.0, 0.3, 2.0):
        for kind, h in (("l1", abs), ("l2sq", lambda v: 0.5 * v * v)):
            got = O.prox_entries(w, kind, t)
            for wi, gi in zip(w, got):
                r = minimize_scalar(lambda v: 0.5 * (v - wi) ** 2 + t * h(v), bounds=(-10, 10), method="bounded",
                                    options={"xatol": 1e-12})
                assert abs(gi - r.x) < 1e-6, (kind, t, wi)
            assert np.all(np.abs(got) <= np.abs(w) + 1e-15) and np.all(got * w >= 0)       # shrinks, keeps the sign
            w2 = w + 0.1 * rng.normal(size=w.shape)
            assert np.linalg.norm(O.prox_entries(w2, kind, t) - got) <= np.linalg.norm(w2 - w) + 1e-15   # non-expansive
    np.testing.assert_array_equal(O.prox_l1(w, 0.0), w)
    assert np.all(O.prox_l1(w, 0.3)[np.abs(w) <= 0.3] == 0.0)                               # the dead zone of the l1 prox
    np.testing.assert_allclose(O.prox_l2sq(w, 1.0), 0.5 * w)
    assert O.prox_entries(w, None, 5.0) is not None and np.array_equal(O.prox_entries(w, None, 5.0), w)
    # a step with a regulariser is the plain step followed by the operator with t = eta * weight
    W, X, y = rng.normal(size=(5, 7)), rng.normal(size=(6, 7)), rng.integers(0, 5, size=6)
    plain = O.sfb_step(O.MLR, W, X, None, y, workers=2, eta=0.2)
    np.testing.assert_array_equal(O.sfb_step(O.MLR, W, X, None, y, workers=2, eta=0.2, prox_kind="l1", prox_weight=0.5),
                                  O.prox_l1(plain, 0.1))
