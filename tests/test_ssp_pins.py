"""Pins of the stale-synchronous emulation oracle (Section 4.1 consistency models; Section 5 reference sequence)."""
import numpy as np

import sfb_inputs as I
from oracle import sfb_oracle as O
from oracle import ssp_oracle as E


def _setup(P=3, B=4, clocks=12, rows=9, cols=7, seed=0):
    wl = I.scaled(I.WORKLOADS["mlr_mid"], "mlr_ssp", rows=rows, cols=cols, workers=P, batch=B, eta=0.2, w_std=0.3,
                  x_scale="unit", seed=seed)
    W0 = I.initial_W(wl)
    batches = []
    for c in range(clocks):
        inp = I.step_inputs(wl, c)
        batches.append([(inp.X[p * B:(p + 1) * B], None, inp.labels[p * B:(p + 1) * B]) for p in range(P)])
    return wl, W0, batches


def test_zero_staleness_is_the_bulk_synchronous_step():
    wl, W0, batches = _setup()
    clocks, P = len(batches), wl.workers
    etas = [0.2] * clocks
    Wp, ref, _ = E.emulate(O.MLR, W0, batches, etas, I.ssp_delays(0, clocks, P, 0), 0)
    W = np.asarray(W0, dtype=np.float64)
    for c in range(clocks):
        inp = I.step_inputs(wl, c)
        # what a replica holds after clock c under BSP: everything up to clock c-1, plus its own update of clock c;
        # after the deliveries of the next clock start, all of clock c.  The reference holds all of clock c.
        W = O.sfb_step(O.MLR, W, inp.X, None, inp.labels, workers=P, eta=0.2)
        np.testing.assert_allclose(ref[c], W, atol=1e-13)
    # one more clock with empty step size delivers the last sets: then every replica is the bulk-synchronous W
    Wp2, ref2, _ = E.emulate(O.MLR, W0, batches + [batches[0]], etas + [0.0], I.ssp_delays(0, clocks + 1, P, 0), 0)
    for p in range(P):
        np.testing.assert_allclose(Wp2[-1][p], W, atol=1e-13)


def test_staleness_guarantee_and_eventual_agreement():
    wl, W0, batches = _setup(clocks=14)
    clocks, P, s = len(batches), wl.workers, 2
    etas = [0.2] * clocks
    # the last s + 1 clocks use step size 0: nothing new is produced while the deliveries under way arrive
    for c in range(clocks - (s + 1), clocks):
        etas[c] = 0.0
    delays = I.ssp_delays(3, clocks, P, s)
    assert delays.max() == s and delays.min() == 0
    Wp, ref, seen = E.emulate(O.MLR, W0, batches, etas, delays, s)
    stale_somewhere = False
    for c in range(clocks):
        for p in range(P):
            must = {(c0, q) for c0 in range(0, c - s) for q in range(P)} | {(c0, p) for c0 in range(c + 1)}
            assert must <= seen[c][p], (c, p)                                   # the guarantee of Section 4.1
            stale_somewhere |= len(seen[c][p]) < (c + 1) * P
    assert stale_somewhere                                                      # the schedule really was stale
    for p in range(P):
        np.testing.assert_allclose(Wp[-1][p], ref[-1], atol=1e-12)              # same sets, only their order differs


def test_asynchronous_execution_agrees_once_every_set_has_arrived():
    """No bound on the delays (Section 4.1, asynchronous parallel): once every factor set has reached every worker all
    replicas hold W_0 plus the same sets, so they equal the reference whatever the order of arrival."""
    wl, W0, batches = _setup(clocks=30)
    clocks, P = len(batches), wl.workers
    delays = I.asp_delays(5, clocks, P, 2.5)
    assert delays.max() >= 6                                   # really beyond any small staleness bound
    tail = int(delays.max()) + 1
    etas = [0.2] * (clocks - tail) + [0.0] * tail              # nothing new while the deliveries under way arrive
    delays[clocks - tail:] = 0
    Wp, ref, seen = E.emulate(O.MLR, W0, batches, etas, delays, None)
    late = max(c - c0 for c in range(clocks) for p in range(P) for c0 in range(c)
               if any((c0, q) not in seen[c][p] for q in range(P)))
    assert late >= 4                                           # some worker ran four or more clocks behind another
    for p in range(P):
        np.testing.assert_allclose(Wp[-1][p], ref[-1], atol=1e-12)


def test_distance_to_the_reference_decays_with_a_decreasing_step_size():
    wl, W0, batches = _setup(clocks=60, seed=1)
    clocks, P, s = len(batches), wl.workers, 3
    etas = [0.5 / (c + 1) for c in range(clocks)]
    Wp, ref, _ = E.emulate(O.MLR, W0, batches, etas, I.ssp_delays(4, clocks, P, s), s)
    dist = [max(np.linalg.norm(Wp[c][p] - ref[c]) for p in range(P)) for c in range(clocks)]
    assert max(dist[:10]) > 0
    assert max(dist[-10:]) < 0.1 * max(dist[:10])                               # Theorem 1: the replicas close in
