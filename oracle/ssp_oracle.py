"""CPU oracle of sufficient-factor broadcasting under bounded staleness.  TEST INFRASTRUCTURE, not a product path.

Section 4.1 (consistency models): under stale synchronous parallel (SSP) with staleness s, a worker at clock c is
guaranteed to have applied every worker's updates of clocks <= c - s - 1, and may have applied some fresher ones;
its own updates it always sees.  s = 0 is bulk-synchronous execution.  Section 5 (Theorem 1) compares each worker's
replica W_p^c with the reference sequence W^c that applies every update in clock order, and shows that their distance
vanishes for a decreasing step size.

Asynchronous parallel execution (the third model named there) puts no bound on the delay: staleness = None
accepts any non-negative delays.

Emulated here exactly as stated, in fp64 numpy: P replicas; at clock c each worker first applies the factor sets
whose delivery is due, then computes the factors of its minibatch against ITS replica, applies them to its own
replica at once with the step eta_c, and posts them to every other worker q with the delivery clock
c + 1 + delay[c][p][q], 0 <= delay <= s (the delays are inputs).  A set is applied with the step size of the clock that
produced it.  Readings: a worker applies deliveries in (clock, sender) order; the reference applies the sets of a
clock in sender order at the end of that clock.

Pins (tests/test_ssp_pins.py): s = 0 reproduces the bulk-synchronous step of oracle.sfb_oracle clock by clock; the SSP
guarantee holds by bookkeeping at every clock; after all deliveries every replica equals the reference (also without a
bound on the delays); with eta_c = eta_0 / (c + 1) the largest distance to the reference decays.
"""
from __future__ import annotations

import numpy as np

from . import sfb_oracle as O


def emulate(model, W0, batches, etas, delays, staleness, margin=1.0, lam=0.1, L=None, iters=20):
    """batches[c][p] = (X, Y, labels) of worker p at clock c; etas[c]; delays[c][p][q].
    Returns (replicas[c][p] after clock c, reference[c] after clock c, seen[c][p] = set of (clock, sender) applied)."""
    clocks, P = len(batches), len(batches[0])
    W = [np.asarray(W0, dtype=np.float64).copy() for _ in range(P)]
    ref = np.asarray(W0, dtype=np.float64).copy()
    inbox = [[] for _ in range(P)]                     # (due, clock, sender, U, V)
    seen = [set() for _ in range(P)]
    out_W, out_ref, out_seen = [], [], []
    for c in range(clocks):
        produced = []
        for p in range(P):
            due = sorted([m for m in inbox[p] if m[0] <= c], key=lambda m: (m[1], m[2]))
            inbox[p] = [m for m in inbox[p] if m[0] > c]
            for _, c0, q, U, V in due:
                W[p] = O.rank_k_update(W[p], U, V, etas[c0])
                seen[p].add((c0, q))
            X, Y, labels = batches[c][p]
            U, V = O.worker_factors(model, W[p], X, Y, labels, margin, lam, L, iters)
            W[p] = O.rank_k_update(W[p], U, V, etas[c])
            seen[p].add((c, p))
            produced.append((U, V))
            for q in range(P):
                if q != p:
                    assert 0 <= delays[c][p][q] and (staleness is None or delays[c][p][q] <= staleness)
                    inbox[q].append((c + 1 + int(delays[c][p][q]), c, p, U, V))
        for p in range(P):
            ref = O.rank_k_update(ref, produced[p][0], produced[p][1], etas[c])
        out_W.append([w.copy() for w in W])
        out_ref.append(ref.copy())
        out_seen.append([set(s) for s in seen])
    return out_W, out_ref, out_seen

