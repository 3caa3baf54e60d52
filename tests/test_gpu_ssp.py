"""Bounded-staleness execution on the GPU (P logical workers, each with its own replica and context, factor sets
delivered late through sfb_set_factors) against the oracle's emulation of Section 4.1 with the same delay schedule:
every replica at every clock, the reference sequence, and the agreement of all replicas once every set has arrived."""
import numpy as np
import pytest

import paper_1409_5705_b200 as S
import sfb_inputs as I
from oracle import sfb_oracle as O
from oracle import ssp_oracle as E
from paper_1409_5705_b200.consistency import StaleSynchronousWorkers
from _parity import to_dev

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def _run(model_name, prec, s, clocks, tol, asp_mean=0.0):
    P, B = 3, 8
    if model_name == "mlr":
        wl = I.scaled(I.WORKLOADS["mlr_mid"], "mlr_ssp", rows=45, cols=36, workers=P, batch=B, eta=0.2, w_std=0.3,
                      x_scale="unit")
    else:
        wl = I.scaled(I.WORKLOADS["dml"], "dml_ssp", rows=24, cols=40, workers=P, batch=B, eta=2e-3)
    W0 = I.initial_W(wl)
    etas = [wl.eta / (c + 1) for c in range(clocks)]
    if asp_mean > 0.0:                                        # asynchronous: no bound on the delays (s is None)
        delays = I.asp_delays(7, clocks, P, asp_mean)
        tail = int(delays.max()) + 1
        delays[clocks - tail:] = 0
    else:
        delays = I.ssp_delays(7, clocks, P, s)
        tail = s + 1
    for c in range(clocks - tail, clocks):
        etas[c] = 0.0                                         # let the deliveries under way arrive
    batches_h = []
    for c in range(clocks):
        inp = I.step_inputs(wl, c)
        batches_h.append([(inp.X[p * B:(p + 1) * B], None if inp.Y is None else inp.Y[p * B:(p + 1) * B],
                           inp.labels[p * B:(p + 1) * B]) for p in range(P)])
    Wp_ref, seq_ref, _ = E.emulate(wl.model, W0, batches_h, etas, delays, s, margin=wl.dml_margin)
    one = I.scaled(wl, "one", workers=1)
    Ws = [to_dev(W0, torch) for _ in range(P + 1)]
    ctxs = [S.Context(S.make_config(one.model, one.rows, one.cols, 1, B, wl.eta, prec, dml_margin=wl.dml_margin), W)
            for W in Ws]
    run = StaleSynchronousWorkers(ctxs[:P], ctxs[P])
    worst = 0.0
    for c in range(clocks):
        run.clock([tuple(to_dev(a, torch) for a in b) for b in batches_h[c]], etas[c], delays[c])
        scale = np.linalg.norm(seq_ref[c] - W0)
        for p in range(P):
            worst = max(worst, np.linalg.norm(Ws[p].cpu().numpy() - Wp_ref[c][p]) / scale)
        worst = max(worst, np.linalg.norm(Ws[P].cpu().numpy() - seq_ref[c]) / scale)
    for ctx in ctxs:
        assert ctx.sfb_get_status() == 0
        ctx.close()
    print(f"{model_name} staleness {s}: worst replica error over {clocks} clocks {worst:.2e} (tol {tol})")
    assert worst <= tol
    # what is still queued was produced in the last s + 1 clocks, whose step size is 0: it would change nothing
    final = [w.cpu().numpy().astype(np.float64) for w in Ws]
    for p in range(P):                                        # every set has arrived: the replicas agree with the reference
        assert np.linalg.norm(final[p] - final[P]) <= 10 * tol * np.linalg.norm(final[P] - W0)


def test_mlr_fp32_bulk_synchronous_and_stale():
    _run("mlr", S.PREC_FP32, 0, 8, 2e-5)
    _run("mlr", S.PREC_FP32, 2, 12, 2e-5)


def test_mlr_fp32_asynchronous():
    _run("mlr", S.PREC_FP32, None, 24, 2e-5, asp_mean=2.0)


def test_dml_split_bf16_stale():
    _run("dml", S.PREC_BF16, 2, 10, 2e-4)


def test_mlr_bf16_stale():
    """The default precision: a worker sends the fp32 u formed from its logits (sfb_export_factors), the receiver splits
    it again into bf16 operand and fp32 class entry."""
    _run("mlr", S.PREC_BF16, 2, 10, 4e-3)


def test_export_and_receive_call_order_and_refusals():
    W = torch.zeros((16, 8), dtype=torch.float32, device="cuda")
    U = torch.zeros((4, 16), dtype=torch.float32, device="cuda")
    V = torch.zeros((4, 8), dtype=torch.float32, device="cuda")
    ctx = S.Context(S.make_config(S.MLR, 16, 8, 1, 4, 0.1, S.PREC_BF16), W)
    with pytest.raises(S.SfbError) as e:                      # nothing computed yet: nothing to send
        ctx.sfb_export_factors(0, U, V)
    assert e.value.code == -9
    ctx.close()
    ctx = S.Context(S.make_config(S.L2MLR, 16, 8, 1, 4, 0.1, S.PREC_FP32, sdca_lambda=0.1, sdca_n=32), W)
    with pytest.raises(S.SfbError) as e:                      # the dual step has no receiving side here
        ctx.sfb_set_factors(0, U, V)
    assert e.value.code == -10
    ctx.close()
