"""A whole step launched as one CUDA graph (the launch-bound small workloads: seven to fifty kernels of a few
microseconds each): captured from the same library calls, the replays give bit-identical results to eager launches."""
import numpy as np
import pytest

import paper_1409_5705_b200 as S
import sfb_inputs as I
from oracle import sfb_oracle as O
from _parity import TOL, config_for, oracle_step, rel_err, to_dev

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")

CASES = {
    "mlr": (I.scaled(I.WORKLOADS["mlr_mid"], "mlr_graph", rows=333, cols=260, workers=3, batch=37, eta=0.05, w_std=0.05,
                     x_scale="unit"), S.PREC_BF16),
    "dml": (I.scaled(I.WORKLOADS["dml"], "dml_graph", rows=150, cols=388, workers=4, batch=33, eta=1e-3), S.PREC_BF16),
    "sc": (I.scaled(I.WORKLOADS["sc"], "sc_graph", rows=300, cols=200, workers=3, batch=11, eta=1e-2, sc_nnz=6), S.PREC_FP32),
}


@pytest.mark.parametrize("name", sorted(CASES))
def test_graph_replays_equal_eager_steps(name):
    wl, prec = CASES[name]
    W0 = I.initial_W(wl)
    L = float(np.float32(O.lipschitz_power_iteration(W0))) if wl.model == I.SC else 0.0
    inps = [I.step_inputs(wl, t) for t in range(2)]
    side = torch.cuda.Stream()
    results = []
    for graphed in (False, True):
        with torch.cuda.stream(side):
            W = to_dev(W0, torch)
            ctx = S.Context(config_for(wl, prec, L), W, stream=side)
            dev = [(to_dev(i.X, torch), to_dev(i.Y, torch), to_dev(i.labels, torch)) for i in inps]
            ctx.sfb_step(*dev[0])                                     # one-off set-up happens in an eager step
            side.synchronize()
            W.copy_(to_dev(W0, torch))
            ctx.sfb_refresh_operands()
            if graphed:
                steps = [ctx.capture(lambda d=d: ctx.sfb_step(*d)) for d in dev]
                W.copy_(to_dev(W0, torch))                            # captures do not run anything
                ctx.sfb_refresh_operands()
                for g in steps:
                    g.replay()
            else:
                for d in dev:
                    ctx.sfb_step(*d)
            side.synchronize()
            assert ctx.sfb_get_status() == 0
            assert ctx.sfb_get_stats().steps >= 2
            results.append(W.cpu().numpy())
            ctx.close()
    assert np.array_equal(results[0], results[1])
    ref = oracle_step(wl, W0, inps[0], L=L if wl.model == I.SC else None)
    ref = oracle_step(wl, ref, inps[1], L=L if wl.model == I.SC else None)
    assert rel_err(results[1], ref, W0) <= 5 * TOL[prec]          # two free-running steps
