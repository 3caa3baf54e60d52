"""Update-only parity: the reconstruct-and-apply pass on its own, onto W = 0.

One step normally ends in W_0 + dW stored in fp32, where the rounding of the sum hides errors of dW that are small
against W_0.  Here the factors are computed against the real W_0, then the caller zeroes W (it owns that buffer)
before sfb_apply_update, so what the pass leaves in W is the update matrix -eta * sum_i u_i v_i^T itself and the
stated tolerances (1e-5 with fp32 operands, 2e-3 with bf16 operands) test the product with no storage floor."""
import numpy as np
import pytest

import paper_1409_5705_b200 as S
import sfb_inputs as I
from oracle import sfb_oracle as O
from _parity import TOL, config_for, to_dev

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")

PRECS = [pytest.param(S.PREC_FP32, id="fp32"), pytest.param(S.PREC_BF16, id="bf16")]
CASES = {
    "mlr": I.scaled(I.WORKLOADS["mlr_mid"], "mlr_upd", rows=333, cols=260, workers=3, batch=37, eta=0.05, w_std=0.05,
                    x_scale="unit"),
    "mlr_mid": I.WORKLOADS["mlr_mid"],
    "dml": I.scaled(I.WORKLOADS["dml"], "dml_upd", rows=150, cols=388, workers=4, batch=33, eta=1e-3),
    "dml_full": I.WORKLOADS["dml"],
    "sc": I.scaled(I.WORKLOADS["sc"], "sc_upd", rows=300, cols=200, workers=3, batch=11, eta=1e-2, sc_nnz=6),
}


@pytest.mark.parametrize("prec", PRECS)
@pytest.mark.parametrize("name", sorted(CASES))
def test_update_matrix_alone_meets_the_stated_tolerance(name, prec):
    wl = CASES[name]
    W0 = I.initial_W(wl)
    inp = I.step_inputs(wl, 0)
    L = float(np.float32(O.lipschitz_power_iteration(W0))) if wl.model == I.SC else 0.0
    W = to_dev(W0, torch)
    ctx = S.Context(config_for(wl, prec, L, prox=0), W)
    ctx.sfb_compute_factors(-1, to_dev(inp.X, torch), to_dev(inp.Y, torch), to_dev(inp.labels, torch))
    ctx.sfb_gather_factors()
    W.zero_()                                   # same stream: ordered after the factors, before the update
    ctx.sfb_apply_update()
    assert ctx.sfb_get_status() == 0
    dW = W.cpu().numpy().astype(np.float64)
    ctx.close()
    _, U, V = O.sfb_step(wl.model, W0, inp.X, inp.Y, inp.labels, workers=wl.workers, eta=wl.eta,
                         margin=wl.dml_margin, lam=wl.sc_lambda, L=L if wl.model == I.SC else None,
                         iters=wl.sc_iters, prox=False, return_factors=True)
    ref = -wl.eta * (U.T @ V)
    err = np.linalg.norm(dW - ref) / np.linalg.norm(ref)
    print(f"{name}: update-only rel err {err:.3e} (tol {TOL[prec]})")
    assert err <= TOL[prec]
    # entry-wise: nothing is absorbed by a large W, so every entry is held to the tolerance, relative to its own size
    # plus 16 rms entries of its row of the update (the rows of frequent classes of MLR sum a hundred terms a hundred
    # times the matrix rms, and an fp32 accumulator rounds relative to what it holds)
    rms = np.sqrt((ref * ref).mean())
    rms_row = np.maximum(np.sqrt((ref * ref).mean(axis=1, keepdims=True)), rms)
    assert ((np.abs(dW - ref) - TOL[prec] * np.abs(ref)) / rms_row).max() <= 16 * TOL[prec]
