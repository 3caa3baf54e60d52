"""Failure detection on the device, in its harmless form: the bounded wait that every tensor-core pipeline stage uses
is made to run out on a barrier nothing arrives at (a one-block kernel with no copy in flight and no tensor memory),
and the host must see SFB_STATUS_TIMEOUT while the context stays usable.  No GPU fault, trap or endless loop is
involved: the wait has a cycle limit and the kernel returns normally."""
import time

import numpy as np
import pytest

import paper_1409_5705_b200 as S
import sfb_inputs as I
from _parity import TOL, config_for, oracle_step, rel_err, to_dev

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def test_a_wait_that_runs_out_sets_the_timeout_bit_and_the_context_stays_usable():
    wl = I.scaled(I.WORKLOADS["mlr_mid"], "mlr_wait", rows=300, cols=260, workers=2, batch=40, w_std=0.05,
                  x_scale="unit")
    W0 = I.initial_W(wl)
    inp = I.step_inputs(wl, 0)
    W = to_dev(W0, torch)
    ctx = S.Context(config_for(wl, S.PREC_BF16), W)
    assert ctx.sfb_get_status() == 0
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    ctx.sfb_selftest_wait_timeout(1_000_000)                 # about half a millisecond of SM cycles
    status = ctx.sfb_get_status()                            # synchronises the stream
    dt = time.perf_counter() - t0
    assert status & S.STATUS_TIMEOUT, f"status word {status:#x}"
    assert dt < 0.010, f"the bounded wait took {dt * 1e3:.2f} ms to give up"
    assert ctx.sfb_get_status() == 0                         # reading the word cleared it
    # the next ordinary step on the same context is clean and correct
    ctx.sfb_step(to_dev(inp.X, torch), None, to_dev(inp.labels, torch))
    assert ctx.sfb_get_status() == 0
    ref = oracle_step(wl, W0, inp)
    assert rel_err(W.cpu().numpy(), ref, W0) <= TOL[S.PREC_BF16]
    with pytest.raises(S.SfbError):
        ctx.sfb_selftest_wait_timeout(0)                     # limits outside 1 .. 2e9 cycles are refused
    ctx.close()
