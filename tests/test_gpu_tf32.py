"""fp32 mode on the tensor cores (every fp32 value as a pair of tf32 words, three products per term) against the
oracle at the fp32 tolerance, on ragged small shapes (forced with PREC_TF32X3) and at a full-size workload (chosen by
PREC_FP32 itself), and against the FFMA kernels of the same mode."""
import numpy as np
import pytest

import paper_1409_5705_b200 as S
import sfb_inputs as I
from oracle import sdca_oracle as D
from _parity import TOL, config_for, entries_ok, oracle_step, rel_err, to_dev

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")
TOL32 = TOL[S.PREC_FP32]


def _small():
    return I.scaled(I.WORKLOADS["mlr_mid"], "mlr_tf32", rows=333, cols=260, workers=3, batch=37, eta=0.05, w_std=0.05,
                    x_scale="unit")


def _step(wl, W0, inp, prec, per_worker=False):
    W = to_dev(W0, torch)
    ctx = S.Context(config_for(wl, prec), W)
    X, lab = to_dev(inp.X, torch), to_dev(inp.labels, torch)
    if per_worker:
        B = wl.batch
        for p in reversed(range(wl.workers)):
            ctx.sfb_compute_factors(p, X[p * B:(p + 1) * B], None, lab[p * B:(p + 1) * B])
        ctx.sfb_gather_factors()
        ctx.sfb_apply_update()
    else:
        ctx.sfb_step(X, None, lab)
    U, V = ctx.factors_as_tensors()
    out = W.cpu().numpy(), U.cpu().numpy(), V.cpu().numpy(), ctx.sfb_get_status(), ctx.sfb_get_stats().last_loss
    ctx.close()
    return out


def test_small_ragged_step_on_the_tensor_cores_meets_the_fp32_tolerance():
    wl = _small()
    W0, inp = I.initial_W(wl), I.step_inputs(wl, 0)
    ref, Uref, Vref = oracle_step(wl, W0, inp, return_factors=True)
    W, U, V, st, loss = _step(wl, W0, inp, S.PREC_TF32X3)
    assert st == 0
    err = rel_err(W, ref, W0)
    print(f"tf32x3 small: rel err {err:.3e} (tol {TOL32})")
    assert err <= TOL32
    assert np.abs(U - Uref).max() <= 2e-6 and np.array_equal(V, inp.X)
    Wf, _, _, _, lossf = _step(wl, W0, inp, S.PREC_FP32_FFMA)
    assert rel_err(Wf, ref, W0) <= TOL32 and abs(loss - lossf) <= 1e-5
    Ww, _, _, st, _ = _step(wl, W0, inp, S.PREC_TF32X3, per_worker=True)
    assert st == 0 and np.array_equal(Ww, W)                 # per-worker calls, any order: the same bits


def test_fp32_mode_picks_the_tensor_cores_at_full_size_and_several_steps_stay_within_tolerance():
    wl = I.WORKLOADS["mlr_mid"]
    W0 = I.initial_W(wl)
    W = to_dev(W0, torch)
    ctx = S.Context(config_for(wl, S.PREC_FP32), W)
    Wt = W0
    for t in range(2):
        inp = I.step_inputs(wl, t)
        ctx.sfb_step(to_dev(inp.X, torch), None, to_dev(inp.labels, torch))
        assert ctx.sfb_get_status() == 0
        Wg = W.cpu().numpy()
        ref = oracle_step(wl, Wt, inp)
        err = rel_err(Wg, ref, Wt)
        print(f"mlr_mid fp32 (tensor cores) step {t}: rel err {err:.3e}")
        assert err <= TOL32
        bulk = np.setdiff1d(np.arange(wl.rows), inp.labels)
        assert entries_ok(Wg[bulk], ref[bulk], Wt[bulk], TOL32)
        Wt = Wg
    flops = ctx.sfb_get_stats().flops
    assert flops > 2 * 2 * (3 + 1) * wl.K * wl.rows * wl.cols * 0.99      # two steps x (3-term forward + update)
    ctx.close()


def test_sdca_on_the_tensor_cores():
    N, J, Dm, P, B, lam = 400, 333, 260, 3, 37, 0.1
    K = P * B
    A = (I.normal_matrix(0, 31, N, Dm, 1.0) * np.float32(3.0 / np.sqrt(Dm))).astype(np.float32)
    y = (np.abs(I.normal_matrix(0, 32, N, 1, 1000.0)[:, 0]).astype(np.int64) % J).astype(np.int32)
    cfg = S.make_config(S.L2MLR, J, Dm, P, B, 1.0 / K, S.PREC_TF32X3, sdca_lambda=lam, sdca_n=N)
    W = torch.zeros((J, Dm), dtype=torch.float32, device="cuda")
    Q = to_dev(D.initial_dual(y, J).astype(np.float32), torch)
    ctx = S.Context(cfg, W)
    ctx.sfb_sdca_set_dual(Q)
    rng = np.random.default_rng(9)
    for step in range(3):
        ids = rng.choice(N, size=K, replace=False).astype(np.int32)
        W_t, Q_t = W.cpu().numpy(), Q.cpu().numpy()
        ctx.sfb_sdca_step(to_dev(A[ids], torch), to_dev(y[ids], torch), to_dev(ids, torch))
        assert ctx.sfb_get_status() == 0
        W_ref, Q_ref, _, _ = D.sdca_step(W_t, A[ids], y[ids], ids, Q_t, lam, 1.0 / K, workers=P)
        err = np.linalg.norm(W.cpu().numpy().astype(np.float64) - W_ref.astype(np.float32)) / np.linalg.norm(W_ref - W_t)
        print(f"sdca tf32x3 step {step}: rel err {err:.3e}")
        assert err <= TOL32 and np.abs(Q.cpu().numpy() - Q_ref).max() <= 2e-6
    ctx.close()


def test_tensor_core_fp32_mode_is_for_the_logistic_models():
    with pytest.raises(S.SfbError) as e:
        S.sfb_workspace_bytes(S.make_config(S.DML, 64, 64, 1, 8, 0.1, S.PREC_TF32X3))
    assert e.value.code == -10


@pytest.mark.parametrize("shape", [(5, 8, 1, 3), (40, 36, 2, 17), (257, 68, 1, 1)])
def test_degenerate_shapes_on_the_tensor_cores(shape):
    """Matrices smaller than one tile, a contraction shorter than one k-block, one sample: everything is padding."""
    rows, cols, P, B = shape
    wl = I.scaled(I.WORKLOADS["mlr_mid"], "mlr_tf32_tiny", rows=rows, cols=cols, workers=P, batch=B, eta=0.1, w_std=0.3,
                  x_scale="unit")
    W0, inp = I.initial_W(wl), I.step_inputs(wl, 0)
    ref = oracle_step(wl, W0, inp)
    W, _, _, st, _ = _step(wl, W0, inp, S.PREC_TF32X3)
    assert st == 0
    assert rel_err(W, ref, W0) <= TOL32
