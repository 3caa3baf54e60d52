"""Sufficient-factor broadcasting over several GPUs: host-side sequencing only.  Two forms:

* ``replica_step`` -- the paper's own (Section 3, Figure 1): every rank holds a full replica of W, computes the
  factors of its logical workers, the ranks all-gather their factors (K*(rows+cols)*4 bytes in total, the linear volume
  of Section 5), and every rank applies all K pairs to its replica.
* ``sharded_step`` -- W partitioned by rows (multiclass logistic regression), described next.

Row-sharded multiclass logistic regression:

Each rank owns a contiguous block of the rows (classes) of W and a block of the K samples of a step (its logical
workers).  One step is

    all-gather of the ranks' samples and class ids          K*cols*4 + K*4 bytes received in total per rank
    sfb_forward_partials on the local rows                  (library kernels)
    all-gather of the per-sample softmax partials           shards*K*16 bytes
    sfb_finish_factors, sfb_gather_factors, sfb_apply_update on the local rows   (library kernels)

so W, U and the update never leave their GPU.  The collectives run through ``torch.distributed`` on whatever backend
the process group has (NCCL on GPUs); no arithmetic happens here.
"""
from __future__ import annotations

from dataclasses import dataclass

from . import MLR, PREC_BF16


def row_shard_bounds(rows: int, shards: int, g: int) -> tuple[int, int]:
    """Rows [r0, r1) of shard g when ``rows`` rows are dealt to ``shards`` shards as evenly as possible (the first
    ``rows % shards`` shards get one row more)."""
    if not (0 <= g < shards) or shards < 1 or rows < shards:
        raise ValueError(f"bad shard {g} of {shards} for {rows} rows")
    base, rem = divmod(rows, shards)
    r0 = g * base + min(g, rem)
    return r0, r0 + base + (1 if g < rem else 0)


@dataclass
class ExchangeBytes:
    """Bytes this rank received in the collectives of one step."""
    samples: int = 0
    partials: int = 0

    @property
    def total(self) -> int:
        return self.samples + self.partials


def exchange_model_bytes(P: int, B: int, rows: int, cols: int, shards: int) -> dict:
    """Values moved per step by the schemes of the paper's cost table (Section 5), in bytes of fp32, for P workers with
    B samples each, beside what the row-sharded step moves: the paper's peer-to-peer broadcast of sufficient factors,
    P*(P-1)*B*(rows+cols); full-matrix synchronisation, P*rows*cols (every worker's update matrix); row sharding,
    per rank the other ranks' samples plus everyone's partials."""
    K = P * B
    return {
        "sfb_p2p": 4 * P * (P - 1) * B * (rows + cols),
        "full_matrix_sync": 4 * P * rows * cols,
        "row_sharded_per_rank": (shards - 1) * (K // shards) * (cols * 4 + 4) + (shards - 1) * K * 16,
    }


def sharded_step(ctx, X_local, labels_local, partials, partials_all, X_all, labels_all, group=None, dist=None,
                 Y_local=None, Y_all=None):
    """One row-sharded step on this rank.

    ctx            a context over this rank's rows, already told its shard with ``sfb_set_row_shard``
    X_local        [K/shards, cols] this rank's samples; labels_local [K/shards] their (global) class ids (MLR) or
                   similar / dissimilar flags (DML)
    partials       scratch for this rank's partials, [K, 4] (MLR) or [K, 1] (DML);  partials_all  [shards, K, 4 | 1]
    X_all          [K, cols] and labels_all [K]: receive the gathered samples (rank-major = worker-major order)
    Y_local, Y_all DML only: the pair partners, gathered like the samples
    dist           the ``torch.distributed`` module (or a stand-in with the same two calls); None: single shard
    Returns the ExchangeBytes of the step.
    """
    moved = ExchangeBytes()
    pairs = Y_local is not None
    if dist is None:
        X_all.copy_(X_local)
        labels_all.copy_(labels_local)
        if pairs:
            Y_all.copy_(Y_local)
    else:
        dist.all_gather_into_tensor(X_all, X_local, group=group)
        dist.all_gather_into_tensor(labels_all, labels_local, group=group)
        moved.samples = (X_all.numel() - X_local.numel()) * X_all.element_size() + \
                        (labels_all.numel() - labels_local.numel()) * labels_all.element_size()
        if pairs:
            dist.all_gather_into_tensor(Y_all, Y_local, group=group)
            moved.samples += (Y_all.numel() - Y_local.numel()) * Y_all.element_size()
    if pairs:
        ctx.sfb_forward_partials_pairs(X_all, Y_all, labels_all, partials)
    else:
        ctx.sfb_forward_partials(X_all, labels_all, partials)
    if dist is None:
        partials_all.view(-1).copy_(partials.view(-1))
    else:
        dist.all_gather_into_tensor(partials_all.view(-1, partials.shape[-1]), partials, group=group)   # shard-major rows
        moved.partials = (partials_all.numel() - partials.numel()) * partials_all.element_size()
    shards = partials_all.shape[0]
    ctx.sfb_finish_factors(partials_all, shards)
    ctx.sfb_gather_factors()
    ctx.sfb_apply_update()
    return moved


def replica_step(ctx, my_workers, X_local, Y_local, labels_local, U_all, V_all, group=None, dist=None):
    """One step of the replica form on this rank.

    ctx          a context over this rank's replica of W with ALL P workers in its config (any precision)
    my_workers   the worker indices this rank computes, ascending and contiguous; X_local [len*B, in_dim] etc. hold
                 their samples in that order
    U_all, V_all [K, rows], [K, cols] fp32: receive every worker's factors (worker-major)
    Returns the bytes this rank received.
    """
    B = ctx.cfg.batch
    for k, p in enumerate(my_workers):
        sl = slice(k * B, (k + 1) * B)
        ctx.sfb_compute_factors(p, X_local[sl], None if Y_local is None else Y_local[sl],
                                None if labels_local is None else labels_local[sl])
    lo, hi = my_workers[0] * B, (my_workers[-1] + 1) * B
    # what this rank sends: its workers' factors in fp32, written straight into their places of the receive buffers
    U_own, V_own = U_all[lo:hi], V_all[lo:hi]
    for k, p in enumerate(my_workers):
        ctx.sfb_export_factors(p, U_own[k * B:(k + 1) * B], V_own[k * B:(k + 1) * B])
    if dist is None:
        received = 0
    else:
        dist.all_gather_into_tensor(U_all, U_own.clone(), group=group)
        dist.all_gather_into_tensor(V_all, V_own.clone(), group=group)
        received = (U_all.numel() - U_own.numel() + V_all.numel() - V_own.numel()) * U_all.element_size()
    mine = set(my_workers)
    # MLR in bf16 mode rounds a received u to its bf16 operand; a rank takes its own factors back the same way, so that
    # every replica applies the same operands bit for bit and the replicas do not drift apart
    reimport_own = getattr(ctx.cfg, "model", None) == MLR and getattr(ctx.cfg, "precision", None) == PREC_BF16
    for q in range(ctx.cfg.workers):
        if q not in mine or reimport_own:
            ctx.sfb_set_factors(q, U_all[q * B:(q + 1) * B], V_all[q * B:(q + 1) * B])
    ctx.sfb_gather_factors()
    ctx.sfb_apply_update()
    return received
