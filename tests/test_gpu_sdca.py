"""GPU parity of the SDCA step of l2-regularised multiclass logistic regression (Section 2.1, "Stochastic DCA")
against the fp64 oracle: the dual rows, the factors and W after mini-batch steps, teacher-forced from the GPU's own
state, on ragged shapes; and a run of sweeps on a small problem whose duality gap the oracle's formulas must see
shrink."""
import numpy as np
import pytest

import paper_1409_5705_b200 as S
import sfb_inputs as I
from oracle import sdca_oracle as D
from _parity import TOL, to_dev

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")

PRECS = [pytest.param(S.PREC_FP32, id="fp32"), pytest.param(S.PREC_BF16, id="bf16")]


def _problem(N, J, Dm, seed):
    """Features ~ N(0,1)/sqrt(D) with the Zipf-free uniform labels of the small MLR workload; seeded inputs only."""
    A = I.normal_matrix(seed, 31, N, Dm, 1.0) * np.float32(1.0 / np.sqrt(Dm)) * np.float32(3.0)
    y = (np.abs(I.normal_matrix(seed, 32, N, 1, 1000.0)[:, 0]).astype(np.int64) % J).astype(np.int32)
    return A.astype(np.float32), y


@pytest.mark.parametrize("prec", PRECS)
def test_minibatch_steps_match_the_oracle_teacher_forced(prec):
    N, J, Dm, P, B, lam = 500, 333, 260, 3, 37, 0.1
    K = P * B
    A, y = _problem(N, J, Dm, 0)
    gamma = 1.0 / K
    cfg = S.make_config(S.L2MLR, J, Dm, P, B, gamma, prec, sdca_lambda=lam, sdca_n=N)
    W = torch.zeros((J, Dm), dtype=torch.float32, device="cuda")
    Q = to_dev(D.initial_dual(y, J).astype(np.float32), torch)
    ctx = S.Context(cfg, W)
    ctx.sfb_sdca_set_dual(Q)
    rng = np.random.default_rng(5)
    for step in range(4):
        ids = rng.choice(N, size=K, replace=False).astype(np.int32)
        W_t, Q_t = W.cpu().numpy(), Q.cpu().numpy()
        if step == 2:                                         # per-worker calls, any order
            for p in reversed(range(P)):
                sl = slice(p * B, (p + 1) * B)
                ctx.sfb_sdca_compute_factors(p, to_dev(A[ids[sl]], torch), to_dev(y[ids[sl]], torch), to_dev(ids[sl], torch))
            ctx.sfb_gather_factors()
            ctx.sfb_apply_update()
        else:
            ctx.sfb_sdca_step(to_dev(A[ids], torch), to_dev(y[ids], torch), to_dev(ids, torch))
        assert ctx.sfb_get_status() == 0
        W_ref, Q_ref, U_ref, _ = D.sdca_step(W_t, A[ids], y[ids], ids, Q_t, lam, gamma, workers=P)
        den = np.linalg.norm(W_ref - W_t)
        err = np.linalg.norm(W.cpu().numpy().astype(np.float64) - W_ref.astype(np.float32)) / den
        errq = np.abs(Q.cpu().numpy() - Q_ref).max()
        print(f"step {step}: W rel err {err:.3e} (tol {TOL[prec]}), dual rows max abs err {errq:.2e}")
        assert err <= TOL[prec]
        assert errq <= (2e-6 if prec == S.PREC_FP32 else 2e-5)  # bf16 mode: logits from bf16 operands, solve in fp32
        rows_sum = Q.cpu().numpy().astype(np.float64).sum(axis=1)
        assert np.abs(rows_sum - 1).max() < 1e-5
    ctx.close()


def test_sweeps_shrink_the_duality_gap():
    """fp32 operands, single-sample steps (K = 1, eta = 1) swept over a small training set: the oracle's primal and
    dual objectives, evaluated on the GPU's W and Q, must close the gap, and W must stay the W of the dual state."""
    N, J, Dm, lam = 40, 12, 24, 0.1
    A, y = _problem(N, J, Dm, 1)
    cfg = S.make_config(S.L2MLR, J, Dm, 1, 1, 1.0, S.PREC_FP32, sdca_lambda=lam, sdca_n=N)
    W = torch.zeros((J, Dm), dtype=torch.float32, device="cuda")
    Q = to_dev(D.initial_dual(y, J).astype(np.float32), torch)
    ctx = S.Context(cfg, W)
    ctx.sfb_sdca_set_dual(Q)
    Ad, yd = to_dev(A, torch), to_dev(y, torch)
    idd = torch.arange(N, dtype=torch.int32, device="cuda")
    gaps = []
    for sweep in range(25):
        for i in range(N):
            ctx.sfb_sdca_step(Ad[i:i + 1], yd[i:i + 1], idd[i:i + 1])
        Wh, Qh = W.cpu().numpy(), Q.cpu().numpy().astype(np.float64)
        Qh = np.clip(Qh, 0, None)
        Qh /= Qh.sum(axis=1, keepdims=True)
        gaps.append(D.l2mlr_primal(Wh, A, y, lam) + D.l2mlr_dual(Qh, A, y, lam))
    assert ctx.sfb_get_status() == 0
    print("duality gap per sweep:", " ".join(f"{g:.2e}" for g in gaps[::4]))
    assert gaps[0] < np.log(J) and gaps[-1] < 1e-5 and gaps[-1] < 1e-3 * gaps[0]
    np.testing.assert_allclose(W.cpu().numpy(), D.w_from_dual(Q.cpu().numpy(), A, y, lam), atol=2e-5)
    ctx.close()


def test_sdca_argument_and_state_errors():
    cfg = S.make_config(S.L2MLR, 16, 8, 1, 4, 0.25, S.PREC_FP32, sdca_lambda=0.1, sdca_n=10)
    W = torch.zeros((16, 8), dtype=torch.float32, device="cuda")
    ctx = S.Context(cfg, W)
    X = torch.zeros((4, 8), dtype=torch.float32, device="cuda")
    lab = torch.zeros(4, dtype=torch.int32, device="cuda")
    ids = torch.tensor([0, 1, 2, 99], dtype=torch.int32, device="cuda")
    with pytest.raises(S.SfbError) as e:
        ctx.sfb_sdca_step(X, lab, ids)                         # no dual state yet
    assert e.value.code == -9
    with pytest.raises(S.SfbError) as e:
        ctx.sfb_step(X, None, lab)                             # the plain step cannot serve a dual context
    assert e.value.code == -10
    Q = torch.zeros((10, 16), dtype=torch.float32, device="cuda")
    Q[:, 0] = 1.0
    ctx.sfb_sdca_set_dual(Q)
    ctx.sfb_sdca_step(X, lab, ids)
    assert ctx.sfb_get_status() & S.STATUS_SAMPLE_RANGE         # id 99 of 10 was skipped and flagged
    ctx.close()
    bad = S.make_config(S.L2MLR, 16, 8, 1, 4, 0.25, S.PREC_FP32, sdca_lambda=0.0, sdca_n=10)
    with pytest.raises(S.SfbError):
        S.sfb_workspace_bytes(bad)
    plain = S.Context(S.make_config(S.MLR, 16, 8, 1, 4, 0.25, S.PREC_FP32), W)
    with pytest.raises(S.SfbError) as e:
        plain.sfb_sdca_step(X, lab, ids)
    assert e.value.code == -10
    plain.close()


def test_a_sample_without_features_moves_its_dual_row_to_the_softmax_and_leaves_W_alone():
    """a_i = 0: kappa = 0, the coordinate problem has no quadratic term and its minimiser is softmax(z) = softmax(0),
    the uniform distribution; the factor pair (du_i, 0) changes nothing in W."""
    N, J, Dm = 8, 20, 12
    cfg = S.make_config(S.L2MLR, J, Dm, 1, 2, 1.0, S.PREC_FP32, sdca_lambda=0.1, sdca_n=N)
    W = torch.zeros((J, Dm), dtype=torch.float32, device="cuda")
    y = np.array([3, 7], dtype=np.int32)
    Q = to_dev(D.initial_dual(np.arange(N) % J, J).astype(np.float32), torch)
    ctx = S.Context(cfg, W)
    ctx.sfb_sdca_set_dual(Q)
    X = torch.zeros((2, Dm), dtype=torch.float32, device="cuda")
    ctx.sfb_sdca_step(X, to_dev(y, torch), to_dev(np.array([3, 7], dtype=np.int32), torch))
    assert ctx.sfb_get_status() == 0
    Qh = Q.cpu().numpy()
    np.testing.assert_allclose(Qh[3], np.full(J, 1.0 / J), atol=1e-6)
    np.testing.assert_allclose(Qh[7], np.full(J, 1.0 / J), atol=1e-6)
    assert float(W.abs().max()) == 0.0
    ctx.close()
