"""Host-side logic of the row-sharded step, without a GPU: the shard bounds, the byte model, and the sequencing of
``sharded_step`` on two gloo ranks with a stand-in context whose three calls do, in numpy fp64, what include/sfb.h
says the library calls do.  The result of the two ranks together must be the oracle's unsharded step."""
import os
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
torch = pytest.importorskip("torch")


def test_shard_bounds_partition_the_rows():
    from paper_1409_5705_b200.sharded import row_shard_bounds
    for rows, G in [(333, 2), (333, 3), (325_000, 8), (10, 10), (1000, 7)]:
        b = [row_shard_bounds(rows, G, g) for g in range(G)]
        assert b[0][0] == 0 and b[-1][1] == rows
        assert all(b[g][1] == b[g + 1][0] for g in range(G - 1))
        sizes = [r1 - r0 for r0, r1 in b]
        assert max(sizes) - min(sizes) <= 1 and sizes == sorted(sizes, reverse=True)
    with pytest.raises(ValueError):
        row_shard_bounds(3, 4, 0)


def test_byte_model_against_the_counting_oracle():
    from oracle import sfb_oracle as O
    from paper_1409_5705_b200.sharded import exchange_model_bytes
    P, B, rows, cols = 16, 64, 325_000, 10_000
    m = exchange_model_bytes(P, B, rows, cols, 8)
    _, p2p, fms = O.comm_values(rows, cols, P, B)
    assert m["sfb_p2p"] == 4 * p2p
    assert m["full_matrix_sync"] == 4 * fms
    # per rank: the 7 other ranks' 128 samples each (features + class id) and 7 x K partials of 16 bytes
    assert m["row_sharded_per_rank"] == 7 * 128 * (cols * 4 + 4) + 7 * 1024 * 16
    assert m["row_sharded_per_rank"] * 8 < m["sfb_p2p"] / 50


class _FakeShard:
    """What the three C-ABI calls compute for one row shard, in numpy fp64 on CPU tensors (a test double)."""

    def __init__(self, W_shard, row_offset, eta):
        self.W = W_shard.astype(np.float64)
        self.r0 = row_offset
        self.eta = eta
        self.calls = []

    def sfb_forward_partials(self, X_all, labels_all, partials):
        self.calls.append("forward")
        self.X = X_all.numpy().astype(np.float64)
        self.y = labels_all.numpy().astype(np.int64)
        self.z = self.X @ self.W.T
        m = self.z.max(axis=1)
        s = np.exp(self.z - m[:, None]).sum(axis=1)
        yl = self.y - self.r0
        mine = (yl >= 0) & (yl < self.W.shape[0])
        zy = np.where(mine, self.z[np.arange(len(yl)), np.clip(yl, 0, self.W.shape[0] - 1)], 0.0)
        partials.copy_(torch.from_numpy(np.stack([m, s, zy, mine.astype(np.float64)], axis=1)))

    def sfb_finish_factors(self, partials_all, shards):
        self.calls.append("finish")
        p = partials_all.numpy().astype(np.float64)
        assert p.shape[0] == shards
        M = p[:, :, 0].max(axis=0)
        lse = M + np.log((p[:, :, 1] * np.exp(p[:, :, 0] - M)).sum(axis=0))
        self.u = np.exp(self.z - lse[:, None])
        yl = self.y - self.r0
        for i, j in enumerate(yl):
            if 0 <= j < self.W.shape[0]:
                self.u[i, j] -= 1.0

    def sfb_gather_factors(self):
        self.calls.append("gather")

    def sfb_apply_update(self):
        self.calls.append("update")
        self.W -= self.eta * (self.u.T @ self.X)


def _rank_main(rank, world, port, out_dir):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import sfb_inputs as I
    from paper_1409_5705_b200.sharded import row_shard_bounds, sharded_step
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    wl = I.scaled(I.WORKLOADS["mlr_mid"], "mlr_gloo", rows=45, cols=24, workers=4, batch=5, eta=0.05, w_std=0.05,
                  x_scale="unit")
    W0 = I.initial_W(wl)
    inp = I.step_inputs(wl, 0)
    K, n = wl.K, wl.K // world
    r0, r1 = row_shard_bounds(wl.rows, world, rank)
    ctx = _FakeShard(W0[r0:r1], r0, wl.eta)
    X_local = torch.from_numpy(inp.X[rank * n:(rank + 1) * n].astype(np.float64))      # this rank's logical workers
    y_local = torch.from_numpy(inp.labels[rank * n:(rank + 1) * n])
    partials = torch.zeros((K, 4), dtype=torch.float64)
    partials_all = torch.zeros((world, K, 4), dtype=torch.float64)
    X_all = torch.zeros((K, wl.cols), dtype=torch.float64)
    y_all = torch.zeros((K,), dtype=y_local.dtype)
    moved = sharded_step(ctx, X_local, y_local, partials, partials_all, X_all, y_all, dist=dist)
    np.save(os.path.join(out_dir, f"W{rank}.npy"), ctx.W)
    np.save(os.path.join(out_dir, f"moved{rank}.npy"), np.array([moved.samples, moved.partials]))
    assert ctx.calls == ["forward", "finish", "gather", "update"]
    assert np.array_equal(y_all.numpy(), inp.labels)                                  # rank-major = worker-major
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_step_their_row_shards_to_the_oracle_result(tmp_path):
    import torch.multiprocessing as mp
    sys.path.insert(0, ROOT)
    import sfb_inputs as I
    from oracle import sfb_oracle as O
    port = 31500 + os.getpid() % 2000
    mp.spawn(_rank_main, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    wl = I.scaled(I.WORKLOADS["mlr_mid"], "mlr_gloo", rows=45, cols=24, workers=4, batch=5, eta=0.05, w_std=0.05,
                  x_scale="unit")
    W0 = I.initial_W(wl)
    inp = I.step_inputs(wl, 0)
    ref = O.sfb_step(O.MLR, W0, inp.X, None, inp.labels, workers=wl.workers, eta=wl.eta)
    W = np.concatenate([np.load(tmp_path / f"W{r}.npy") for r in range(2)], axis=0)
    assert np.linalg.norm(W - ref) <= 1e-12 * np.linalg.norm(ref - W0)
    moved = np.load(tmp_path / "moved0.npy")
    K = wl.K
    assert moved[0] == (K // 2) * wl.cols * 8 + (K // 2) * inp.labels.itemsize          # the other rank's samples (fp64 here)
    assert moved[1] == K * 4 * 8                                                       # the other rank's partials


def test_single_shard_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import sfb_inputs as I
    from oracle import sfb_oracle as O
    from paper_1409_5705_b200.sharded import sharded_step
    wl = I.scaled(I.WORKLOADS["mlr_mid"], "mlr_one", rows=17, cols=12, workers=2, batch=3, eta=0.1, w_std=0.05,
                  x_scale="unit")
    W0 = I.initial_W(wl)
    inp = I.step_inputs(wl, 0)
    ctx = _FakeShard(W0, 0, wl.eta)
    K = wl.K
    moved = sharded_step(ctx, torch.from_numpy(inp.X.astype(np.float64)), torch.from_numpy(inp.labels),
                         torch.zeros((K, 4), dtype=torch.float64), torch.zeros((1, K, 4), dtype=torch.float64),
                         torch.zeros((K, wl.cols), dtype=torch.float64), torch.zeros((K,), dtype=torch.int32))
    ref = O.sfb_step(O.MLR, W0, inp.X, None, inp.labels, workers=wl.workers, eta=wl.eta)
    assert np.linalg.norm(ctx.W - ref) <= 1e-12 * np.linalg.norm(ref - W0)
    assert moved.total == 0


class _FakeReplica:
    """What the calls of the replica form do, in numpy fp64 (a test double): factors of a worker from the oracle's own
    formula for MLR, factors taken from elsewhere, and the update with all of them."""

    class _Cfg:
        pass

    def __init__(self, W, P, B, eta):
        from oracle import sfb_oracle as O
        self.O = O
        self.W = W.astype(np.float64)
        self.cfg = self._Cfg()
        self.cfg.workers, self.cfg.batch = P, B
        self.eta = eta
        self.U = torch.zeros((P * B, W.shape[0]), dtype=torch.float64)
        self.V = torch.zeros((P * B, W.shape[1]), dtype=torch.float64)
        self.have = set()

    def sfb_compute_factors(self, p, X, Y, labels):
        B = self.cfg.batch
        U, V = self.O.mlr_factors(self.W, X.numpy(), labels.numpy())
        self.U[p * B:(p + 1) * B] = torch.from_numpy(U)
        self.V[p * B:(p + 1) * B] = torch.from_numpy(V)
        self.have.add(p)

    def sfb_export_factors(self, p, U_out, V_out):
        B = self.cfg.batch
        U_out.copy_(self.U[p * B:(p + 1) * B])
        V_out.copy_(self.V[p * B:(p + 1) * B])

    def sfb_set_factors(self, q, U, V):
        B = self.cfg.batch
        self.U[q * B:(q + 1) * B] = U
        self.V[q * B:(q + 1) * B] = V
        self.have.add(q)

    def sfb_gather_factors(self):
        assert self.have == set(range(self.cfg.workers))

    def sfb_apply_update(self):
        self.W = self.O.rank_k_update(self.W, self.U.numpy(), self.V.numpy(), self.eta)


def _replica_rank(rank, world, port, out_dir):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import sfb_inputs as I
    from paper_1409_5705_b200.sharded import replica_step
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    wl = I.scaled(I.WORKLOADS["mlr_mid"], "mlr_rep", rows=15, cols=12, workers=4, batch=3, eta=0.1, w_std=0.2,
                  x_scale="unit")
    W0 = I.initial_W(wl)
    inp = I.step_inputs(wl, 0)
    B, K = wl.batch, wl.K
    mine = [2 * rank, 2 * rank + 1]
    lo, hi = mine[0] * B, (mine[-1] + 1) * B
    ctx = _FakeReplica(W0, wl.workers, B, wl.eta)
    U_all = torch.zeros((K, wl.rows), dtype=torch.float64)
    V_all = torch.zeros((K, wl.cols), dtype=torch.float64)
    got = replica_step(ctx, mine, torch.from_numpy(inp.X[lo:hi].astype(np.float64)), None, torch.from_numpy(inp.labels[lo:hi]),
                       U_all, V_all, dist=dist)
    np.save(os.path.join(out_dir, f"R{rank}.npy"), ctx.W)
    assert got == (K - 2 * B) * (wl.rows + wl.cols) * 8
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_keep_identical_replicas_equal_to_the_oracle_step(tmp_path):
    import torch.multiprocessing as mp
    sys.path.insert(0, ROOT)
    import sfb_inputs as I
    from oracle import sfb_oracle as O
    port = 33500 + os.getpid() % 2000
    mp.spawn(_replica_rank, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    wl = I.scaled(I.WORKLOADS["mlr_mid"], "mlr_rep", rows=15, cols=12, workers=4, batch=3, eta=0.1, w_std=0.2,
                  x_scale="unit")
    W0 = I.initial_W(wl)
    inp = I.step_inputs(wl, 0)
    ref = O.sfb_step(O.MLR, W0, inp.X, None, inp.labels, workers=wl.workers, eta=wl.eta)
    R0, R1 = np.load(tmp_path / "R0.npy"), np.load(tmp_path / "R1.npy")
    assert np.array_equal(R0, R1)
    assert np.linalg.norm(R0 - ref) <= 1e-12 * np.linalg.norm(ref - W0)


class _FakeDmlShard:
    """The DML calls of one row shard in numpy fp64 (a test double): partial squared norms, hinge on their sum."""

    def __init__(self, W_shard, eta, margin):
        self.W = W_shard.astype(np.float64)
        self.eta, self.margin = eta, margin

    def sfb_forward_partials_pairs(self, X_all, Y_all, similar_all, partials):
        self.v = (X_all.numpy() - Y_all.numpy()).astype(np.float64)
        self.sim = similar_all.numpy()
        self.z = self.v @ self.W.T
        partials.copy_(torch.from_numpy((self.z * self.z).sum(axis=1, keepdims=True)))

    def sfb_finish_factors(self, partials_all, shards):
        q = partials_all.numpy().astype(np.float64).sum(axis=0)[:, 0]
        c = np.where(self.sim != 0, 2.0, np.where(q < self.margin, -2.0, 0.0))
        self.u = c[:, None] * self.z

    def sfb_gather_factors(self):
        pass

    def sfb_apply_update(self):
        self.W -= self.eta * (self.u.T @ self.v)


def _dml_workload():
    import sfb_inputs as I
    return I.scaled(I.WORKLOADS["dml"], "dml_gloo", rows=14, cols=20, workers=4, batch=5, eta=1e-2, dml_margin=0.8)


def _dml_rank(rank, world, port, out_dir):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import sfb_inputs as I
    from paper_1409_5705_b200.sharded import row_shard_bounds, sharded_step
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    wl = _dml_workload()
    W0 = I.initial_W(wl)
    inp = I.step_inputs(wl, 0)
    K, n = wl.K, wl.K // world
    r0, r1 = row_shard_bounds(wl.rows, world, rank)
    ctx = _FakeDmlShard(W0[r0:r1], wl.eta, wl.dml_margin)
    sl = slice(rank * n, (rank + 1) * n)
    f64 = lambda a: torch.from_numpy(a.astype(np.float64))
    partials = torch.zeros((K, 1), dtype=torch.float64)
    partials_all = torch.zeros((world, K, 1), dtype=torch.float64)
    X_all, Y_all = torch.zeros((K, wl.cols), dtype=torch.float64), torch.zeros((K, wl.cols), dtype=torch.float64)
    s_all = torch.zeros((K,), dtype=torch.int32)
    moved = sharded_step(ctx, f64(inp.X[sl]), torch.from_numpy(inp.labels[sl]), partials, partials_all, X_all, s_all, dist=dist,
                         Y_local=f64(inp.Y[sl]), Y_all=Y_all)
    np.save(os.path.join(out_dir, f"D{rank}.npy"), ctx.W)
    assert moved.samples == 2 * (K - n) * wl.cols * 8 + (K - n) * 4 and moved.partials == K * 8
    assert np.array_equal(Y_all.numpy(), inp.Y.astype(np.float64))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_step_dml_row_shards_to_the_oracle_result(tmp_path):
    import torch.multiprocessing as mp
    sys.path.insert(0, ROOT)
    import sfb_inputs as I
    from oracle import sfb_oracle as O
    port = 33500 + os.getpid() % 2000
    mp.spawn(_dml_rank, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    wl = _dml_workload()
    W0 = I.initial_W(wl)
    inp = I.step_inputs(wl, 0)
    ref = O.sfb_step(O.DML, W0, inp.X, inp.Y, inp.labels, workers=wl.workers, eta=wl.eta, margin=wl.dml_margin)
    W = np.concatenate([np.load(tmp_path / f"D{r}.npy") for r in range(2)], axis=0)
    assert np.linalg.norm(W - ref) <= 1e-12 * np.linalg.norm(ref - W0)
    assert np.linalg.norm(ref - W0) > 0
