"""Entry-wise proximal operators fused into the update pass (proximal SGD, Section 2.1: W <- prox_{eta h}(W - eta dW))
against the oracle: l1 (soft threshold) and squared l2 (shrink), every model, both precisions, and the dense
full-matrix-synchronisation path.  The error is measured against the size of the un-regularised update: both
operators are non-expansive, so they cannot hide an error of the update, and entries that end within rounding of the
l1 dead zone are 0 on one side and ~1e-9 on the other, which this metric rightly ignores."""
import numpy as np
import pytest

import paper_1409_5705_b200 as S
import sfb_inputs as I
from oracle import sfb_oracle as O
from _parity import TOL, storage_floor, to_dev

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")

PRECS = [pytest.param(S.PREC_FP32, id="fp32"), pytest.param(S.PREC_BF16, id="bf16")]
KINDS = [pytest.param((S.PROX_L1, "l1", 0.2), id="l1"), pytest.param((S.PROX_L2SQ, "l2sq", 5.0), id="l2sq")]
CASES = {
    "mlr": I.scaled(I.WORKLOADS["mlr_mid"], "mlr_prox", rows=333, cols=260, workers=3, batch=37, eta=0.05, w_std=0.05,
                    x_scale="unit"),
    "dml": I.scaled(I.WORKLOADS["dml"], "dml_prox", rows=150, cols=388, workers=4, batch=33, eta=1e-3),
    "sc": I.scaled(I.WORKLOADS["sc"], "sc_prox", rows=300, cols=200, workers=3, batch=11, eta=1e-2, sc_nnz=6),
}


def _config(wl, prec, kind, weight, L):
    return S.make_config(wl.model, wl.rows, wl.cols, wl.workers, wl.batch, wl.eta, prec, dml_margin=wl.dml_margin,
                         sc_lambda=wl.sc_lambda, sc_ista_iters=wl.sc_iters, sc_lipschitz=float(L),
                         sc_prox=1 if wl.model == I.SC else 0, prox_kind=kind, prox_weight=weight)


@pytest.mark.parametrize("prec", PRECS)
@pytest.mark.parametrize("kind", KINDS)
@pytest.mark.parametrize("name", sorted(CASES))
def test_step_with_an_entrywise_prox_matches_the_oracle(name, kind, prec):
    wl = CASES[name]
    code, oname, weight = kind
    if wl.model != I.MLR:
        weight *= 20.0                                   # eta is 1e-3 .. 1e-2 there: keep the operator visible
    W0 = I.initial_W(wl)
    inp = I.step_inputs(wl, 0)
    L = float(np.float32(O.lipschitz_power_iteration(W0))) if wl.model == I.SC else 0.0
    W = to_dev(W0, torch)
    ctx = S.Context(_config(wl, prec, code, weight, L), W)
    ctx.sfb_step(to_dev(inp.X, torch), to_dev(inp.Y, torch), to_dev(inp.labels, torch))
    assert ctx.sfb_get_status() == 0
    Wg = W.cpu().numpy().astype(np.float64)
    ctx.close()
    kw = dict(workers=wl.workers, eta=wl.eta, margin=wl.dml_margin, lam=wl.sc_lambda, L=L if wl.model == I.SC else None,
              iters=wl.sc_iters)
    ref = O.sfb_step(wl.model, W0, inp.X, inp.Y, inp.labels, prox=(wl.model == I.SC), prox_kind=oname, prox_weight=weight, **kw)
    plain = O.sfb_step(wl.model, W0, inp.X, inp.Y, inp.labels, prox=False, **kw)
    den = np.linalg.norm(plain - W0)
    err = np.linalg.norm(Wg - ref.astype(np.float32)) / den
    floor = np.linalg.norm(ref.astype(np.float32) - ref) / den
    moved = np.linalg.norm(ref - plain) / den
    print(f"{name} {oname}: err {err:.3e} of the plain update (tol {TOL[prec]}, storage floor {floor:.1e}); the operator "
          f"itself moves W by {moved:.1f} update sizes")
    assert moved > 0.01                                  # the operator really acted
    assert err <= TOL[prec] + (3.0 * floor if wl.model == I.SC else floor)
    if oname == "l1":
        zero_ref = ref == 0.0
        assert zero_ref.mean() > 0.02 and (Wg[zero_ref] == 0.0).mean() > 0.999     # the dead zone is exactly zero


def test_dense_sync_path_applies_the_same_operator():
    wl = CASES["mlr"]
    W0 = I.initial_W(wl)
    inp = I.step_inputs(wl, 0)
    out = []
    for dense in (False, True):
        W = to_dev(W0, torch)
        ctx = S.Context(_config(wl, S.PREC_FP32, S.PROX_L1, 0.2, 0.0), W)
        X, lab = to_dev(inp.X, torch), to_dev(inp.labels, torch)
        if dense:
            ctx.sfb_dense_sync_step(X, None, lab, torch.empty(2 * wl.rows * wl.cols, dtype=torch.float32, device="cuda"))
        else:
            ctx.sfb_step(X, None, lab)
        out.append(W.cpu().numpy().astype(np.float64))
        ctx.close()
    plain = O.sfb_step(wl.model, W0, inp.X, None, inp.labels, workers=wl.workers, eta=wl.eta)
    assert np.linalg.norm(out[0] - out[1]) / np.linalg.norm(plain - W0) <= 2e-5


def test_prox_arguments_are_checked():
    with pytest.raises(S.SfbError):
        S.sfb_workspace_bytes(S.make_config(S.MLR, 16, 8, 1, 4, 0.1, prox_kind=3))
    with pytest.raises(S.SfbError):
        S.sfb_workspace_bytes(S.make_config(S.MLR, 16, 8, 1, 4, 0.1, prox_kind=1, prox_weight=-1.0))
    with pytest.raises(S.SfbError) as e:
        S.sfb_workspace_bytes(S.make_config(S.L2MLR, 16, 8, 1, 4, 0.1, sdca_lambda=0.1, sdca_n=8, prox_kind=1))
    assert e.value.code == -10
