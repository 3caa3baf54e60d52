"""Edge cases of the CUDA path against the oracle: degenerate sizes (one sample, one worker, matrices smaller than
one tile, a contraction shorter than one k-block), degenerate data (every sample of one class, zero W, eta = 0) and
shapes whose every dimension is ragged against every tile size."""
import numpy as np
import pytest

import paper_1409_5705_b200 as S
import sfb_inputs as I
from oracle import sfb_oracle as O
from _parity import TOL, step_tol, config_for, oracle_step, rel_err, to_dev

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")

PRECS = [pytest.param(S.PREC_FP32, id="fp32"), pytest.param(S.PREC_BF16, id="bf16")]


def run_step(wl, W0, inp, prec, L=0.0):
    W = to_dev(W0, torch)
    ctx = S.Context(config_for(wl, prec, L), W)
    ctx.sfb_step(to_dev(inp.X, torch), to_dev(inp.Y, torch), to_dev(inp.labels, torch))
    st = ctx.sfb_get_status()
    out = W.cpu().numpy()
    ctx.close()
    return out, st


def make(name, **kw):
    base = {"mlr": "mlr_mid", "dml": "dml", "sc": "sc"}[name]
    d = dict(x_scale="unit") if name == "mlr" else {}
    d.update(kw)
    return I.scaled(I.WORKLOADS[base], name + "_edge", **d)


SHAPES = [
    # (model, rows, cols, P, B): smaller than any tile; one pair only; K not a multiple of 8 or 64
    ("mlr", 5, 8, 1, 1), ("mlr", 33, 4, 1, 7), ("mlr", 257, 516, 5, 13), ("mlr", 1, 64, 2, 3),
    ("mlr", 333, 260, 2, 150), ("mlr", 700, 132, 1, 256),      # several sample tiles, the last one ragged
    ("dml", 3, 12, 1, 1), ("dml", 129, 260, 3, 5),
    ("sc", 8, 4, 1, 1), ("sc", 261, 132, 2, 9),
]


@pytest.mark.parametrize("prec", PRECS)
@pytest.mark.parametrize("name,rows,cols,P,B", SHAPES)
def test_degenerate_and_ragged_shapes(name, rows, cols, P, B, prec):
    kw = dict(rows=rows, cols=cols, workers=P, batch=B, eta=0.05)
    if name == "mlr":
        kw["w_std"] = 0.05
    if name == "sc":
        kw.update(sc_nnz=min(3, cols), eta=1e-2)
    wl = make(name, **kw)
    W0 = I.initial_W(wl)
    if name == "dml":
        W0 = (W0 * np.float32(0.3)).astype(np.float32)
    inp = I.step_inputs(wl, 0, I.sc_true_dictionary(wl) if name == "sc" else None)
    L = O.lipschitz_power_iteration(W0) if name == "sc" else 0.0
    if name == "dml" and O.dml_hinge_distance(W0, inp.X, inp.Y, inp.labels) < 4e-3:
        pytest.skip("a pair sits on the hinge's kink: two answers are correct")
    ref = oracle_step(wl, W0, inp, L=L)
    Wg, st = run_step(wl, W0, inp, prec, L)
    assert st == 0
    den = np.linalg.norm(ref - W0.astype(np.float64))
    if den == 0:
        np.testing.assert_array_equal(Wg, W0)
    else:
        assert rel_err(Wg, ref, W0) <= step_tol(wl, prec, ref, W0)


@pytest.mark.parametrize("prec", PRECS)
def test_every_sample_of_one_class(prec):
    """All K labels equal: the exact label-row term sums K samples into one row."""
    wl = make("mlr", rows=70, cols=132, workers=2, batch=40, eta=0.05, w_std=0.05)
    W0, inp = I.initial_W(wl), I.step_inputs(wl, 0)
    inp.labels[:] = 69
    ref = oracle_step(wl, W0, inp)
    Wg, st = run_step(wl, W0, inp, prec)
    assert st == 0 and rel_err(Wg, ref, W0) <= TOL[prec]


@pytest.mark.parametrize("prec", PRECS)
@pytest.mark.parametrize("name", ["mlr", "dml", "sc"])
def test_eta_zero_leaves_W_bit_identical(name, prec):
    wl = make(name, rows=140, cols=260, workers=2, batch=20, eta=0.0, **({"sc_nnz": 4} if name == "sc" else {}))
    W0 = I.initial_W(wl)
    if name == "sc":
        W0 = (W0 * np.float32(0.5)).astype(np.float32)          # column norms 0.5: the prox leaves them alone
    inp = I.step_inputs(wl, 0, I.sc_true_dictionary(wl) if name == "sc" else None)
    L = O.lipschitz_power_iteration(W0) if name == "sc" else 0.0
    Wg, st = run_step(wl, W0, inp, prec, L)
    assert st == 0
    np.testing.assert_array_equal(Wg, W0)


def test_zero_matrix_mlr_matches_the_closed_form_in_bf16():
    """W = 0: p = 1/J for every class, so dW = (1/J) 1 (sum x)^T - sum e_y x^T; 1/J with J = 64 is exact in bf16."""
    wl = I.WORKLOADS["mlr_tiny"]
    W0, inp = I.initial_W(wl), I.step_inputs(wl, 0)
    X = inp.X.astype(np.float64)
    dW = np.tile(X.sum(axis=0) / wl.rows, (wl.rows, 1))
    np.subtract.at(dW, inp.labels, X)
    ref = -wl.eta * dW
    Wg, st = run_step(wl, W0, inp, S.PREC_BF16)
    assert st == 0
    assert np.linalg.norm(Wg - ref) / np.linalg.norm(ref) <= TOL[S.PREC_BF16]


@pytest.mark.parametrize("prec", [pytest.param(S.PREC_BF16, id="bf16"), pytest.param(S.PREC_TF32X3, id="tf32x3")])
def test_caller_writes_to_W_between_steps_need_a_refresh_of_the_operand_copy(prec):
    """MLR keeps an operand copy of W for the forward product (bf16, or the pair of tf32 words of the tensor-core
    fp32 mode).  The library keeps it current through its own
    updates; after the CALLER rewrites W, sfb_refresh_operands brings it up to date: the next step is then the oracle's
    step from the new W.  Without the refresh the forward runs on the old copy, which this test also shows."""
    wl = I.scaled(I.WORKLOADS["mlr_mid"], "mlr_refresh", rows=300, cols=260, workers=2, batch=64, eta=0.05,
                  w_std=0.05, x_scale="unit")
    W0 = I.initial_W(wl)
    W1 = (-3.0 * W0).astype(np.float32)                       # what the caller loads over W after step 0
    inp0, inp1 = I.step_inputs(wl, 0), I.step_inputs(wl, 1)
    ref = oracle_step(wl, W1, inp1)
    errs = {}
    tol = TOL[S.PREC_BF16] if prec == S.PREC_BF16 else TOL[S.PREC_FP32]
    for refresh in (True, False):
        W = to_dev(W0, torch)
        ctx = S.Context(config_for(wl, prec), W)
        ctx.sfb_step(to_dev(inp0.X, torch), None, to_dev(inp0.labels, torch))
        W.copy_(torch.from_numpy(W1))                          # the caller's own write to W
        if refresh:
            ctx.sfb_refresh_operands()
        ctx.sfb_step(to_dev(inp1.X, torch), None, to_dev(inp1.labels, torch))
        assert ctx.sfb_get_status() == 0
        errs[refresh] = rel_err(W.cpu().numpy(), ref, W1)
        ctx.close()
    assert errs[True] <= tol, errs
    assert errs[False] > 10 * TOL[S.PREC_BF16], errs           # the stale copy gives another step altogether
