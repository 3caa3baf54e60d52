"""CPU oracle for l2-regularised multiclass logistic regression learnt by stochastic dual coordinate ascent, the
fourth model of the paper.  TEST INFRASTRUCTURE, not a product path: only tests, the smoke check and the bench's
CPU-baseline leg may call it; the CUDA library never does and shares no code with it.  fp64 numpy throughout.

What the paper fixes (Section 2.1, "Stochastic DCA"; Section 3; Section 6):

    (P)  min_W  1/N sum_i f_i(W a_i) + h(W)          f_i(z) = log sum_j exp z_j - z_{y_i},   h(W) = lam/2 ||W||_F^2
    (D)  min_U  1/N sum_i f_i^*(-u_i) + h^*(1/N U A^T)
    W = grad h^*(Z),   Z = 1/N U A^T;     per sample:  u_i <- u_i - du_i,   Z <- Z - du_i a_i^T,   W <- grad h^*(Z)

with du_i the change that minimises (D) over u_i, the other dual vectors held fixed.  The sufficient factors of the
step are (du_i, a_i).  For these f and h (conjugates worked out by hand):

    f_i^*(-u) = sum_j q_j log q_j  with  q = e_{y_i} - u  in the probability simplex (infinite outside it),
    h^*(Z) = ||Z||_F^2 / (2 lam),   grad h^*(Z) = Z / lam,   so   W = 1/(lam N) sum_i (e_{y_i} - q_i) a_i^T.

The dual state is kept as Q [N x J], q_i = e_{y_i} - u_i (u_i = 0, i.e. q_i = e_{y_i}, at the start: W = 0).

Readings where the paper is silent or inconsistent:
 1. The exact coordinate minimiser.  With z = W a_i (W including sample i's current contribution) and
    kappa = ||a_i||^2 / (lam N), minimising (D) over q_i on the simplex is
        min_q  sum_j q_j log q_j - q.(z + kappa q_old) + kappa/2 ||q||^2,
    whose stationarity conditions are   log q_j + kappa q_j = z_j + kappa q_old_j - nu,   sum_j q_j = 1.
    Each coordinate is a Lambert-W expression of nu; nu is found by bisection on [lse(t) - kappa, lse(t)],
    t = z + kappa q_old (the sum of the q_j(nu) is >= 1 at the left end and <= 1 at the right end).
 2. The paper writes Z <- Z - du_i a_i^T; Z = 1/N U A^T changes by -1/N du_i a_i^T.  The 1/N is kept here, so
    that W = grad h^*(Z) stays exactly the W of the dual state: W <- W - gamma/(lam N) sum_i du_i a_i^T.
 3. Mini-batches (Section 3, "Mini-batch proximal SGD/SDCA": the K updates are averaged, 1/K sum u_i v_i^T): every
    sample of the batch solves its coordinate problem against the same W (bulk-synchronous), and the K changes
    are applied with the weight gamma, u_i <- u_i - gamma du_i; gamma = 1/K is the paper's average and keeps (D)
    non-increasing by convexity; gamma = 1 with K = 1 is the single-sample step of Section 2.1.
 4. du_i is "the stochastic update" subtracted from u_i:  du_i = u_old - u_new = q_new - q_old.

Pins (tests/test_sdca_pins.py): the coordinate minimiser against scipy's bounded minimiser and against an
independent one-dimensional root for two classes; its kappa -> 0 limit softmax(z); weak duality (P + D >= 0) for
arbitrary feasible Q; monotone decrease of (D) for single-sample and averaged mini-batch steps; the incrementally
updated W equal to the W of the dual state; the duality gap going to zero and W reaching the primal optimum that
scipy's L-BFGS finds for (P); the fixed point q = softmax(W a) at that optimum.
"""
from __future__ import annotations

import numpy as np
from scipy.special import lambertw


def _f64(a):
    return np.asarray(a, dtype=np.float64)


def _lse(Z):
    m = Z.max(axis=-1, keepdims=True)
    return (m + np.log(np.exp(Z - m).sum(axis=-1, keepdims=True)))[..., 0]


def l2mlr_primal(W, A, y, lam):
    """(P): 1/N sum_i (log sum_j exp z_ij - z_{i,y_i}) + lam/2 ||W||^2,  z_i = W a_i.  A is [N x D]."""
    W, A = _f64(W), _f64(A)
    Z = A @ W.T
    return float(np.mean(_lse(Z) - Z[np.arange(A.shape[0]), np.asarray(y, dtype=np.int64)]) + 0.5 * lam * np.sum(W * W))


def w_from_dual(Q, A, y, lam):
    """W = grad h^*(Z) = Z / lam with Z = 1/N U A^T and u_i = e_{y_i} - q_i."""
    Q, A = _f64(Q), _f64(A)
    N = A.shape[0]
    U = -Q.copy()
    U[np.arange(N), np.asarray(y, dtype=np.int64)] += 1.0
    return (U.T @ A) / (lam * N)


def l2mlr_dual(Q, A, y, lam):
    """(D): 1/N sum_i sum_j q_ij log q_ij + ||Z||^2 / (2 lam)   (0 log 0 = 0)."""
    Q, A = _f64(Q), _f64(A)
    ent = np.where(Q > 0, Q * np.log(np.where(Q > 0, Q, 1.0)), 0.0).sum()
    Z = lam * w_from_dual(Q, A, y, lam)
    return float(ent / A.shape[0] + np.sum(Z * Z) / (2.0 * lam))


def _coordinates(t, nu, kappa):
    """q_j solving log q_j + kappa q_j = t_j - nu."""
    c = t - nu
    if kappa == 0.0:
        return np.exp(c)
    return lambertw(kappa * np.exp(c)).real / kappa


def coordinate_minimiser(z, q_old, kappa, iters=200):
    """argmin over the simplex of  sum q log q - q.(z + kappa q_old) + kappa/2 ||q||^2   (reading 1)."""
    z, q_old = _f64(z), _f64(q_old)
    t = z + kappa * q_old
    hi = float(_lse(t))                       # sum_j q_j(hi) <= 1
    lo = hi - kappa                           # sum_j q_j(lo) >= 1
    for _ in range(iters):
        mid = 0.5 * (lo + hi)
        if _coordinates(t, mid, kappa).sum() > 1.0:
            lo = mid
        else:
            hi = mid
    q = _coordinates(t, 0.5 * (lo + hi), kappa)
    return q / q.sum()


def sdca_factors(W, X, y, Q_rows, lam, N):
    """Sufficient factors of K samples against the same W:  U [K x J] with rows du_i = q_new_i - q_old_i, V = X.
    Q_rows [K x J] are the samples' current dual rows."""
    W, X, Q_rows = _f64(W), _f64(X), _f64(Q_rows)
    Z = X @ W.T
    U = np.empty_like(Q_rows)
    for i in range(X.shape[0]):
        kappa = float(X[i] @ X[i]) / (lam * N)
        U[i] = coordinate_minimiser(Z[i], Q_rows[i], kappa) - Q_rows[i]
    return U, X.copy()


def sdca_step(W, X, y, ids, Q, lam, gamma, workers=1):
    """One bulk-synchronous mini-batch step on the samples ``ids`` (distinct) of a training set of N = len(Q):
    every worker computes the factors of its B samples against the same W, the factors are gathered, and
        q_i <- q_i + gamma du_i,      W <- W - gamma/(lam N) sum_i du_i a_i^T.
    Returns (W_new, Q_new, U, V)."""
    W, X, Q = _f64(W), _f64(X), _f64(Q).copy()
    N, K = Q.shape[0], X.shape[0]
    ids = np.asarray(ids, dtype=np.int64)
    assert len(np.unique(ids)) == K, "the samples of a step must be distinct"
    B = K // workers
    assert B * workers == K
    parts = []
    for p in range(workers):
        sl = slice(p * B, (p + 1) * B)
        parts.append(sdca_factors(W, X[sl], np.asarray(y)[sl], Q[ids[sl]], lam, N))
    U = np.concatenate([f[0] for f in parts], axis=0)
    V = np.concatenate([f[1] for f in parts], axis=0)
    Q[ids] += gamma * U
    W_new = W - (gamma / (lam * N)) * (U.T @ V)
    return W_new, Q, U, V


def initial_dual(y, J):
    """u_i = 0: q_i = e_{y_i}, so that W = 0."""
    y = np.asarray(y, dtype=np.int64)
    Q = np.zeros((len(y), J))
    Q[np.arange(len(y)), y] = 1.0
    return Q
