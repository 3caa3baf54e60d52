"""CPU oracle for one Sufficient-Factor-Broadcasting minibatch step.  TEST INFRASTRUCTURE, not a product path.

A plain, slow, fp64 numpy statement of what the SFB hot path computes, written from the paper's formulas so
that a reader can check it against the paper by eye.  Only the tests, the smoke check and the bench's
CPU-baseline leg may call it; the CUDA library never does, and the two share no code.

Notation (paper, Section 2): W is the J x D parameter matrix (here ``rows x cols``), a_i the vector that
multiplies it, f_i the per-sample loss, and the per-sample stochastic gradient is the outer product u v^T
with u = d f_i / d (W a_i), v = a_i.  One step, for K = P*B samples drawn by P workers of B samples each
(Section 3, "Mini-batch proximal SGD"), is

    W  <-  prox( W - eta * sum_i u_i v_i^T ).

Pins (tests/test_oracle_pins.py): finite differences of each loss, the independently coded dense gradient,
the rank bound, closed forms (zero-init MLR, DML three-matmul form, orthonormal-dictionary ISTA), invariants
(column sums conserved under MLR, ISTA objective non-increasing, prox idempotent), numpy's spectral norm; the
entry-wise proximal operators against scipy's scalar minimiser of their defining problem.
Multi-step trajectories: parity unpinned beyond composing pinned single steps.
"""
from __future__ import annotations

import numpy as np

MLR, DML, SC = 0, 1, 2


def _f64(a):
    return np.asarray(a, dtype=np.float64)


# ----------------------------------------------------------------------------------------------------------
# Multiclass logistic regression (Section 1: u = prediction vector, v = feature vector; Section 2.1:
# u = d f / d (W a)).  The gradient factor is softmax(W x) - onehot(y).
# ----------------------------------------------------------------------------------------------------------
def mlr_factors(W, X, y):
    """U [K x J], V [K x D] for samples X [K x D] with class ids y [K]."""
    W, X = _f64(W), _f64(X)
    Z = X @ W.T                                   # z_i = W x_i
    Z = Z - Z.max(axis=1, keepdims=True)
    Pm = np.exp(Z)
    Pm /= Pm.sum(axis=1, keepdims=True)
    U = Pm
    U[np.arange(X.shape[0]), np.asarray(y, dtype=np.int64)] -= 1.0
    return U, X.copy()


def mlr_loss(W, X, y):
    """f_i = -z_y + log sum_j exp(z_j), one value per sample."""
    W, X = _f64(W), _f64(X)
    Z = X @ W.T
    m = Z.max(axis=1)
    lse = m + np.log(np.exp(Z - m[:, None]).sum(axis=1))
    return lse - Z[np.arange(X.shape[0]), np.asarray(y, dtype=np.int64)]


# ----------------------------------------------------------------------------------------------------------
# Distance metric learning (Section 2: a_i is the difference of the pair; f_i quadratic for a similar pair,
# hinge for a dissimilar one; Section "Experiments": linear-projection parametrisation, W = L^T, k x D).
#   similar:     f = ||W a||^2                 u =  2 W a
#   dissimilar:  f = max(0, margin - ||W a||^2)  u = -2 W a  if ||W a||^2 < margin  else 0
# ----------------------------------------------------------------------------------------------------------
def dml_factors(W, X, Y, similar, margin=1.0):
    W = _f64(W)
    V = _f64(X) - _f64(Y)
    Z = V @ W.T
    q = (Z * Z).sum(axis=1)
    sim = np.asarray(similar) != 0
    s = np.where(sim, 1.0, np.where(q < margin, -1.0, 0.0))
    return 2.0 * s[:, None] * Z, V


def dml_loss(W, X, Y, similar, margin=1.0):
    W = _f64(W)
    V = _f64(X) - _f64(Y)
    Z = V @ W.T
    q = (Z * Z).sum(axis=1)
    return np.where(np.asarray(similar) != 0, q, np.maximum(0.0, margin - q))


def dml_hinge_distance(W, X, Y, similar, margin=1.0):
    """min over dissimilar pairs of | ||W a||^2 - margin |: how far the batch is from the hinge's kink."""
    W = _f64(W)
    Z = (_f64(X) - _f64(Y)) @ W.T
    q = (Z * Z).sum(axis=1)
    d = np.abs(q - margin)[np.asarray(similar) == 0]
    return float(d.min()) if d.size else float("inf")


# ----------------------------------------------------------------------------------------------------------
# Sparse coding (Section 2: W is the dictionary, columns are atoms with ||W_k|| <= 1, a_i the sparse code,
# f_i quadratic; Figure 3: u = W a - x, v = a, prox rescales columns of norm > 1).  The paper leaves the
# coder open; this build fixes it: T ISTA iterations on 1/2||x - W a||^2 + lam ||a||_1 from a = 0, step 1/L.
# ----------------------------------------------------------------------------------------------------------
def soft_threshold(w, t):
    return np.sign(w) * np.maximum(np.abs(w) - t, 0.0)


def ista_codes(W, X, lam, L, iters):
    """Codes [K x A] after ``iters`` ISTA iterations, every sample started from a = 0."""
    W, X = _f64(W), _f64(X)
    A = np.zeros((X.shape[0], W.shape[1]))
    for _ in range(iters):
        R = A @ W.T - X                           # r = W a - x
        G = R @ W                                 # g = W^T r
        A = soft_threshold(A - G / L, lam / L)
    return A


def sc_objective(W, A, X, lam):
    """1/2||x - W a||^2 + lam ||a||_1 per sample."""
    R = _f64(A) @ _f64(W).T - _f64(X)
    return 0.5 * (R * R).sum(axis=1) + lam * np.abs(A).sum(axis=1)


def sc_factors(W, X, lam, L, iters):
    A = ista_codes(W, X, lam, L, iters)
    U = A @ _f64(W).T - _f64(X)
    return U, A


def sc_loss(W, A, X):
    """f_i = 1/2 ||W a_i - x_i||^2 with the code held fixed (the function whose gradient is u v^T)."""
    R = _f64(A) @ _f64(W).T - _f64(X)
    return 0.5 * (R * R).sum(axis=1)


def lipschitz_power_iteration(W, iters=50):
    """L = ||W||_2^2 by power iteration on W^T W from the normalised all-ones vector (Rayleigh quotient)."""
    W = _f64(W)
    b = np.ones(W.shape[1]) / np.sqrt(W.shape[1])
    for _ in range(iters):
        c = W.T @ (W @ b)
        b = c / np.linalg.norm(c)
    return float(b @ (W.T @ (W @ b)))


def prox_unit_columns(W):
    """Projection onto {||W_k||_2 <= 1 for every column k}: rescale only the columns whose norm exceeds 1."""
    W = _f64(W).copy()
    n = np.sqrt((W * W).sum(axis=0))
    big = n > 1.0
    W[:, big] /= n[big]
    return W


# ----------------------------------------------------------------------------------------------------------
# Entry-wise proximal operators of proximal SGD (Section 2: the regulariser h "could be ... l1-, l2-, trace-norm";
# Section 2.1: after W <- W - eta dW the operator prox_{eta h} is applied).  prox_{t h}(w) = argmin_v 1/2 (v - w)^2 + t h(v).
#   h = lam ||W||_1           prox: shrink every entry towards 0 by t = eta*lam, entries within t of 0 become 0
#   h = lam/2 ||W||_F^2       prox: every entry divided by 1 + t, t = eta*lam
# (The trace norm needs the singular value decomposition of W and is not part of this step.)
# ----------------------------------------------------------------------------------------------------------
def prox_l1(W, t):
    W = _f64(W)
    return np.sign(W) * np.maximum(np.abs(W) - t, 0.0)


def prox_l2sq(W, t):
    return _f64(W) / (1.0 + t)


def prox_entries(W, kind, t):
    """kind: None, "l1" or "l2sq"."""
    if kind is None:
        return _f64(W)
    if kind == "l1":
        return prox_l1(W, t)
    if kind == "l2sq":
        return prox_l2sq(W, t)
    raise ValueError(kind)


# ----------------------------------------------------------------------------------------------------------
# Broadcast, reconstruction, update (Section 3, Figure 1)
# ----------------------------------------------------------------------------------------------------------
def gather(factors_per_worker):
    """Concatenate the P workers' (U_p [B x J], V_p [B x D]) in worker order: row i = p*B + b."""
    U = np.concatenate([f[0] for f in factors_per_worker], axis=0)
    V = np.concatenate([f[1] for f in factors_per_worker], axis=0)
    return U, V


def rank_k_update(W, U, V, eta):
    """W - eta * sum_i u_i v_i^T."""
    return _f64(W) - eta * (_f64(U).T @ _f64(V))


def worker_factors(model, W, X, Y=None, labels=None, margin=1.0, lam=0.1, L=None, iters=20):
    if model == MLR:
        return mlr_factors(W, X, labels)
    if model == DML:
        return dml_factors(W, X, Y, labels, margin)
    if model == SC:
        return sc_factors(W, X, lam, L, iters)
    raise ValueError(model)


def sfb_step(model, W, X, Y=None, labels=None, workers=1, eta=1.0, margin=1.0, lam=0.1, L=None, iters=20,
             prox=False, return_factors=False, prox_kind=None, prox_weight=0.0):
    """One BSP step: every worker computes the SFs of its B samples against the same W, the SFs are
    gathered, every pair is reconstructed and applied, then the proximal operator (SC)."""
    K = X.shape[0]
    B = K // workers
    assert B * workers == K
    per_worker = []
    for p in range(workers):
        sl = slice(p * B, (p + 1) * B)
        per_worker.append(worker_factors(model, W, X[sl], None if Y is None else Y[sl],
                                         None if labels is None else labels[sl], margin, lam, L, iters))
    U, V = gather(per_worker)
    Wn = rank_k_update(W, U, V, eta)
    Wn = prox_entries(Wn, prox_kind, eta * prox_weight)           # prox_{eta h} of an entry-wise regulariser, if any
    if prox:
        Wn = prox_unit_columns(Wn)
    return (Wn, U, V) if return_factors else Wn


# ----------------------------------------------------------------------------------------------------------
# Full-matrix synchronisation (Section 3 "SFB vs client-server", Section 5 cost analysis): every worker
# forms its dense update matrix from its own minibatch; the matrices are summed and applied once.
# The per-sample gradients here are coded element by element, independently of the factor routines above.
# ----------------------------------------------------------------------------------------------------------
def dense_gradient(model, W, X, Y=None, labels=None, margin=1.0, codes=None):
    """sum_i d f_i / d W as a dense matrix, from the element-wise derivative of each loss."""
    W = _f64(W)
    J, D = W.shape
    G = np.zeros((J, D))
    for i in range(X.shape[0]):
        if model == MLR:
            x = _f64(X[i])
            z = np.array([float(np.dot(W[j], x)) for j in range(J)])
            e = np.exp(z - z.max())
            p = e / e.sum()
            for j in range(J):
                G[j, :] += (p[j] - (1.0 if j == int(labels[i]) else 0.0)) * x
        elif model == DML:
            a = _f64(X[i]) - _f64(Y[i])
            z = W @ a
            q = float(z @ z)
            if int(labels[i]) != 0:
                c = 2.0
            else:
                c = -2.0 if q < margin else 0.0
            for j in range(J):
                G[j, :] += c * z[j] * a
        elif model == SC:
            a = _f64(codes[i])
            r = W @ a - _f64(X[i])
            for j in range(J):
                G[j, :] += r[j] * a
        else:
            raise ValueError(model)
    return G


def dense_sync_step(model, W, X, Y=None, labels=None, workers=1, eta=1.0, margin=1.0, codes=None,
                    prox=False):
    """FMS-style step: P dense per-worker update matrices, summed at the 'server', applied, then prox."""
    K = X.shape[0]
    B = K // workers
    total = np.zeros(_f64(W).shape)
    for p in range(workers):
        sl = slice(p * B, (p + 1) * B)
        total += dense_gradient(model, W, X[sl], None if Y is None else Y[sl],
                                None if labels is None else labels[sl], margin,
                                None if codes is None else codes[sl])
    Wn = _f64(W) - eta * total
    return prox_unit_columns(Wn) if prox else Wn


# ----------------------------------------------------------------------------------------------------------
# Communication volume (Section 5, cost table): values moved per iteration.
# ----------------------------------------------------------------------------------------------------------
def comm_values(rows, cols, workers, batch):
    """(one gathered copy of all SFs, the paper's peer-to-peer broadcast count, full-matrix sync)."""
    one_copy = workers * batch * (rows + cols)
    p2p = workers * (workers - 1) * batch * (rows + cols)
    fms = workers * rows * cols
    return one_copy, p2p, fms


# ----------------------------------------------------------------------------------------------------------
# Sampled outputs for shapes too large to hold W in fp64 (paper-scale MLR): the same definitions, evaluated
# for a block of classes at a time / for chosen rows of W only.
# ----------------------------------------------------------------------------------------------------------
def mlr_log_partition(W, X, block_rows=16384):
    """log sum_j exp(z_ij) per sample, visiting the classes j block by block (W may be fp32; each block is
    promoted to fp64).  Equal to the one-shot value up to fp64 rounding."""
    X = _f64(X)
    K = X.shape[0]
    m = np.full(K, -np.inf)
    s = np.zeros(K)
    for r0 in range(0, W.shape[0], block_rows):
        Z = X @ _f64(W[r0:r0 + block_rows]).T
        mb = np.maximum(m, Z.max(axis=1))
        s = s * np.exp(m - mb) + np.exp(Z - mb[:, None]).sum(axis=1)
        m = mb
    return m + np.log(s)


def mlr_updated_rows(W_rows, row_ids, X, y, log_partition, eta):
    """Rows ``row_ids`` of W after one MLR step: W_j - eta * sum_i (p_ij - [j = y_i]) x_i."""
    Wr, X = _f64(W_rows), _f64(X)
    Z = X @ Wr.T                                                  # [K x n]
    U = np.exp(Z - np.asarray(log_partition)[:, None])
    U -= (np.asarray(y, dtype=np.int64)[:, None] == np.asarray(row_ids, dtype=np.int64)[None, :])
    return Wr - eta * (U.T @ X)
