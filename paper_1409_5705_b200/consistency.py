"""Sufficient-factor broadcasting under bounded staleness on one GPU: host-side sequencing only.

P logical workers each own a replica of W and a context over it (one worker, B samples).  A clock of worker p is:
apply the factor sets from other workers whose delivery is due (``sfb_set_factors`` + gather + update, with the step
size of the clock that produced them), compute the factors of its own minibatch against its replica
(``sfb_compute_factors``), apply them at once, and post copies of them to every other worker with a delivery clock at
most ``staleness`` clocks beyond the next one.  Staleness 0 is bulk-synchronous execution; Section 4.1 of the paper
gives the guarantee (a worker at clock c has every update of clocks <= c - s - 1), Section 5 the reference sequence the
replicas are compared with.  All arithmetic runs in the library's kernels; this module only moves factor buffers
between contexts and keeps the delivery queues.
"""
from __future__ import annotations


class StaleSynchronousWorkers:
    def __init__(self, contexts, reference_context=None):
        """contexts[p]: a Context with workers = 1 over worker p's replica (any precision).
        reference_context: optional context over a further copy of W that applies every set in clock order."""
        self.ctx = list(contexts)
        self.ref = reference_context
        self.P = len(self.ctx)
        self.inbox = [[] for _ in range(self.P)]           # (due, clock, sender, eta, U, V)
        self.clock_no = 0

    def _apply(self, ctx, eta, U, V):
        ctx.sfb_set_eta(eta)
        ctx.sfb_set_factors(0, U, V)
        ctx.sfb_gather_factors()
        ctx.sfb_apply_update()

    def clock(self, batches, eta, delays):
        """batches[p] = (X, Y, labels) device tensors of worker p; delays[p][q] in [0, staleness]."""
        c = self.clock_no
        produced = []
        for p, ctx in enumerate(self.ctx):
            due = sorted((m for m in self.inbox[p] if m[0] <= c), key=lambda m: (m[1], m[2]))
            self.inbox[p] = [m for m in self.inbox[p] if m[0] > c]
            for _, _, _, eta0, U, V in due:
                self._apply(ctx, eta0, U, V)
            X, Y, labels = batches[p]
            ctx.sfb_set_eta(eta)
            ctx.sfb_compute_factors(0, X, Y, labels)
            U = X.new_empty((ctx.cfg.batch, ctx.cfg.rows))           # the copy that is "sent"
            V = X.new_empty((ctx.cfg.batch, ctx.cfg.cols))
            ctx.sfb_export_factors(0, U, V)
            ctx.sfb_gather_factors()
            ctx.sfb_apply_update()
            produced.append((U, V))
            for q in range(self.P):
                if q != p:
                    self.inbox[q].append((c + 1 + int(delays[p][q]), c, p, eta, U, V))
        if self.ref is not None:
            for U, V in produced:
                self._apply(self.ref, eta, U, V)
        self.clock_no += 1

    def pending(self):
        return sum(len(b) for b in self.inbox)
