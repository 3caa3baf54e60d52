"""Row-sharded multiclass logistic regression on ONE GPU: G shards of W stepped one after the other in one process,
their softmax partials exchanged through the host, against the unsharded oracle step.  (On several GPUs each shard is a
rank and the exchange is an all-gather; the kernels and the C-ABI calls are the ones exercised here.)"""
import numpy as np
import pytest

import paper_1409_5705_b200 as S
import sfb_inputs as I
from oracle import sfb_oracle as O
from paper_1409_5705_b200.sharded import row_shard_bounds
from _parity import TOL, config_for, oracle_step, rel_err, to_dev

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")

PRECS = [pytest.param(S.PREC_FP32, id="fp32"), pytest.param(S.PREC_BF16, id="bf16"),
         pytest.param(S.PREC_TF32X3, id="tf32x3")]


def _workload():
    # ragged on purpose: 333 rows over 2 or 3 shards gives 167/166 and 111/111/111 rows, none a multiple of a tile
    return I.scaled(I.WORKLOADS["mlr_mid"], "mlr_shards", rows=333, cols=260, workers=3, batch=37, eta=0.05,
                    w_std=0.05, x_scale="unit")


def _sharded_step(wl, W0, inp, prec, G, via_host=True):
    """Steps G row shards of W0 through the three sharded calls; returns (W after the step, losses, status words)."""
    K = wl.K
    X, lab = to_dev(inp.X, torch), to_dev(inp.labels, torch)
    ctxs, Ws = [], []
    for g in range(G):
        r0, r1 = row_shard_bounds(wl.rows, G, g)
        Wg = to_dev(W0[r0:r1], torch)
        sub = I.scaled(wl, f"{wl.name}_{g}", rows=r1 - r0)
        ctx = S.Context(config_for(sub, prec), Wg)
        ctx.sfb_set_row_shard(r0, wl.rows)
        ctxs.append(ctx)
        Ws.append(Wg)
    parts = torch.zeros((G, K, 4), dtype=torch.float32, device="cuda")
    for g, ctx in enumerate(ctxs):
        ctx.sfb_forward_partials(X, lab, parts[g])
    if via_host:                                  # the exchange: every shard gets everyone's partials
        parts = parts.cpu().cuda()
    losses, status = [], []
    for ctx in ctxs:
        ctx.sfb_finish_factors(parts, G)
        ctx.sfb_gather_factors()
        ctx.sfb_apply_update()
        status.append(ctx.sfb_get_status())
        losses.append(ctx.sfb_get_stats().last_loss)
        ctx.close()
    return np.concatenate([w.cpu().numpy() for w in Ws], axis=0), parts.cpu().numpy(), losses, status


@pytest.mark.parametrize("prec", PRECS)
@pytest.mark.parametrize("G", [1, 2, 3])
def test_row_shards_match_the_unsharded_oracle_step(prec, G):
    wl = _workload()
    W0 = I.initial_W(wl)
    inp = I.step_inputs(wl, 0)
    ref = oracle_step(wl, W0, inp)
    W, parts, losses, status = _sharded_step(wl, W0, inp, prec, G)
    assert status == [0] * G
    err = rel_err(W, ref, W0)
    print(f"G={G} rel err {err:.3e} (tol {TOL[prec]})")
    assert err <= TOL[prec]
    # merged partials give the oracle's log-partition; every shard reports the same mean loss, the oracle's
    lse_ref = O.mlr_log_partition(W0, inp.X)
    M = parts[:, :, 0].max(axis=0)
    lse = M + np.log((parts[:, :, 1].astype(np.float64) * np.exp(parts[:, :, 0] - M)).sum(axis=0))
    tol_z = 2e-2 if prec == S.PREC_BF16 else 2e-5
    np.testing.assert_allclose(lse, lse_ref, atol=tol_z)
    assert np.all(parts[:, :, 3].sum(axis=0) == 1.0)                # exactly one shard owns each sample's class
    loss_ref = float(np.mean(O.mlr_loss(W0, inp.X, inp.labels))) / 1.0
    for l in losses:
        assert abs(l - losses[0]) <= 1e-6 * abs(losses[0])
        assert abs(l - loss_ref) <= tol_z


def test_one_shard_is_the_unsharded_path():
    wl = _workload()
    W0 = I.initial_W(wl)
    inp = I.step_inputs(wl, 0)
    W_sh, _, _, _ = _sharded_step(wl, W0, inp, S.PREC_BF16, 1, via_host=False)
    W = to_dev(W0, torch)
    ctx = S.Context(config_for(wl, S.PREC_BF16), W)
    ctx.sfb_step(to_dev(inp.X, torch), None, to_dev(inp.labels, torch))
    assert ctx.sfb_get_status() == 0
    ctx.close()
    ref = oracle_step(wl, W0, inp)
    den = np.linalg.norm(ref - W0)
    assert np.linalg.norm(W_sh.astype(np.float64) - W.cpu().numpy()) / den <= 1e-6


def test_row_shards_over_several_steps_teacher_forced():
    """Three steps on three shards: each step is checked from the shards' own W (the bf16 copies of the shards'
    rows, which the update keeps current, feed the next forward product)."""
    wl = _workload()
    G, K = 3, wl.K
    W0 = I.initial_W(wl)
    ctxs, Ws = [], []
    for g in range(G):
        r0, r1 = row_shard_bounds(wl.rows, G, g)
        Wg = to_dev(W0[r0:r1], torch)
        ctx = S.Context(config_for(I.scaled(wl, f"s{g}", rows=r1 - r0), S.PREC_BF16), Wg)
        ctx.sfb_set_row_shard(r0, wl.rows)
        ctxs.append(ctx)
        Ws.append(Wg)
    parts = torch.zeros((G, K, 4), dtype=torch.float32, device="cuda")
    for t in range(3):
        inp = I.step_inputs(wl, t)
        Wt = np.concatenate([w.cpu().numpy() for w in Ws], axis=0)
        X, lab = to_dev(inp.X, torch), to_dev(inp.labels, torch)
        for g, ctx in enumerate(ctxs):
            ctx.sfb_forward_partials(X, lab, parts[g])
        for ctx in ctxs:
            ctx.sfb_finish_factors(parts, G)
            ctx.sfb_gather_factors()
            ctx.sfb_apply_update()
            assert ctx.sfb_get_status() == 0
        ref = oracle_step(wl, Wt, inp)
        W1 = np.concatenate([w.cpu().numpy() for w in Ws], axis=0)
        assert rel_err(W1, ref, Wt) <= TOL[S.PREC_BF16], f"step {t}"
    for ctx in ctxs:
        ctx.close()


def test_row_shard_call_order_and_argument_errors():
    wl = _workload()
    W = to_dev(I.initial_W(wl)[:100], torch)
    ctx = S.Context(config_for(I.scaled(wl, "s", rows=100), S.PREC_FP32), W)
    parts = torch.zeros((1, wl.K, 4), dtype=torch.float32, device="cuda")
    with pytest.raises(S.SfbError) as e:
        ctx.sfb_finish_factors(parts, 1)                       # no forward partials yet
    assert e.value.code == -9
    with pytest.raises(S.SfbError) as e:
        ctx.sfb_set_row_shard(300, 333)                        # rows [300, 400) do not fit 333 classes
    assert e.value.code == -3
    ctx.sfb_set_row_shard(200, 333)
    inp = I.step_inputs(wl, 0)
    lab = inp.labels.copy()
    lab[5] = 400                                               # a class nobody owns
    ctx.sfb_forward_partials(to_dev(inp.X, torch), to_dev(lab, torch), parts[0])
    ctx.sfb_finish_factors(parts, 1)
    assert ctx.sfb_get_status() & S.STATUS_LABEL_RANGE
    ctx.close()
    wd = I.scaled(I.WORKLOADS["sc"], "d", rows=64, cols=64, workers=1, batch=8)
    Wd = to_dev(I.initial_W(wd), torch)
    cd = S.Context(config_for(wd, S.PREC_FP32), Wd)
    with pytest.raises(S.SfbError) as e:
        cd.sfb_set_row_shard(0, 64)
    assert e.value.code == -10
    cd.close()


@pytest.mark.parametrize("name", ["mlr", "mlr_bf16", "dml"])
def test_replica_form_two_ranks_on_one_gpu(name):
    """The paper's own form: two replicas of W, each computes the factors of half of the workers, the factors are
    exchanged (here: copied between the two contexts' buffers, as an all-gather would), both apply all K pairs.  Both
    replicas must end at the oracle's step."""
    from paper_1409_5705_b200.sharded import replica_step
    if name.startswith("mlr"):
        wl, prec = I.scaled(_workload(), "mlr_rep", workers=4, batch=20), S.PREC_BF16 if name == "mlr_bf16" else S.PREC_FP32
    else:
        wl, prec = I.scaled(I.WORKLOADS["dml"], "dml_rep", rows=150, cols=388, workers=4, batch=33, eta=1e-3), S.PREC_BF16
    W0 = I.initial_W(wl)
    inp = I.step_inputs(wl, 0)
    ref = oracle_step(wl, W0, inp)
    G, B, K = 2, wl.batch, wl.K
    Ws = [to_dev(W0, torch) for _ in range(G)]
    ctxs = [S.Context(config_for(wl, prec), W) for W in Ws]
    U_all = torch.zeros((K, wl.rows), dtype=torch.float32, device="cuda")
    V_all = torch.zeros((K, wl.cols), dtype=torch.float32, device="cuda")
    X, Y, lab = to_dev(inp.X, torch), to_dev(inp.Y, torch), to_dev(inp.labels, torch)
    own = [list(range(g * 2, g * 2 + 2)) for g in range(G)]
    # phase 1: every rank computes and publishes its own factors (what the all-gather delivers)
    for g, ctx in enumerate(ctxs):
        lo, hi = own[g][0] * B, (own[g][-1] + 1) * B
        for p in own[g]:
            sl = slice(p * B, (p + 1) * B)
            ctx.sfb_compute_factors(p, X[sl], None if Y is None else Y[sl], lab[sl])
        for p in own[g]:
            ctx.sfb_export_factors(p, U_all[p * B:(p + 1) * B], V_all[p * B:(p + 1) * B])
    if name == "mlr_bf16":
        # what was sent is the fp32 u of Section 2.1, class entry included (the bf16 layout itself holds 0 there)
        Uo, _ = O.mlr_factors(W0, inp.X, inp.labels)
        assert np.abs(U_all.cpu().numpy() - Uo).max() <= 2e-3 * np.abs(Uo).max()
    # phase 2: every rank takes the others' factors and applies all K pairs
    for g, ctx in enumerate(ctxs):
        for q in range(wl.workers):
            if q not in own[g] or name == "mlr_bf16":          # bf16 MLR: own factors go the same way as received ones
                ctx.sfb_set_factors(q, U_all[q * B:(q + 1) * B], V_all[q * B:(q + 1) * B])
        ctx.sfb_gather_factors()
        ctx.sfb_apply_update()
        assert ctx.sfb_get_status() == 0
        assert rel_err(Ws[g].cpu().numpy(), ref, W0) <= TOL[prec], g
        ctx.close()
    assert torch.equal(Ws[0], Ws[1])                         # the replicas stay bit-identical
    # the single-rank form of the helper gives the same step
    W = to_dev(W0, torch)
    ctx = S.Context(config_for(wl, prec), W)
    assert replica_step(ctx, list(range(wl.workers)), X, Y, lab, U_all, V_all) == 0
    assert torch.equal(W, Ws[0])
    ctx.close()


def test_a_shard_that_owns_no_class_of_the_batch():
    """Every class id of the batch lies in the first shard: the other shards contribute softmax mass only, their
    owner flags are all 0, and their rows still receive the (small) update of the non-label classes."""
    wl = _workload()
    W0 = I.initial_W(wl)
    inp = I.step_inputs(wl, 0)
    inp.labels = (inp.labels % 50).astype(np.int32)            # 3 shards of 111 rows: all labels in shard 0
    ref = oracle_step(wl, W0, inp)
    for prec in (S.PREC_FP32, S.PREC_BF16):
        W, parts, losses, status = _sharded_step(wl, W0, inp, prec, 3)
        assert status == [0, 0, 0]
        assert rel_err(W, ref, W0) <= TOL[prec]
        assert parts[0, :, 3].sum() == wl.K and parts[1:, :, 3].sum() == 0
        assert np.abs(W[111:] - W0[111:]).max() > 0            # the other shards' rows moved too


@pytest.mark.parametrize("G", [1, 2, 3])
@pytest.mark.parametrize("prec", [pytest.param(S.PREC_FP32, id="fp32"), pytest.param(S.PREC_BF16, id="bf16")])
def test_dml_row_shards_match_the_unsharded_oracle_step(prec, G):
    """DML with the latent rows of W dealt to G contexts: every shard computes its part of z = W (x - y) and its
    partial ||z||^2, the partials are exchanged (here through one device buffer), every shard decides the hinge on the
    summed norm and updates its rows.  Both hinge branches occur in the batch."""
    from paper_1409_5705_b200.sharded import sharded_step
    wl = I.scaled(I.WORKLOADS["dml"], "dml_shard", rows=150, cols=388, workers=4, batch=33, eta=1e-3)
    W0 = I.initial_W(wl)
    inp = I.step_inputs(wl, 0)
    zq = ((inp.X - inp.Y).astype(np.float64) @ W0.astype(np.float64).T)
    # the margin near the median norm of the dissimilar pairs: about half of them inside the hinge, half outside
    qs = np.sort((zq * zq).sum(axis=1)[inp.labels == 0])
    mid = len(qs) // 2
    k = max(range(mid - 5, mid + 5), key=lambda t: qs[t + 1] - qs[t])          # the widest gap near the middle: no pair
    wl = I.scaled(wl, "dml_shard_m", dml_margin=float(0.5 * (qs[k] + qs[k + 1])))    # sits on the margin itself
    ref = oracle_step(wl, W0, inp)
    K = wl.K
    X, Y, lab = to_dev(inp.X, torch), to_dev(inp.Y, torch), to_dev(inp.labels, torch)
    parts_all = torch.zeros((G, K, 1), dtype=torch.float32, device="cuda")
    shards = []
    for g in range(G):
        r0, r1 = row_shard_bounds(wl.rows, G, g)
        Wg = to_dev(W0[r0:r1], torch)
        cfg = S.make_config(S.DML, r1 - r0, wl.cols, wl.workers, wl.batch, wl.eta, prec, dml_margin=wl.dml_margin)
        ctx = S.Context(cfg, Wg)
        ctx.sfb_set_row_shard(r0, wl.rows)
        ctx.sfb_forward_partials_pairs(X, Y, lab, parts_all[g])
        shards.append((ctx, Wg))
    q = parts_all.sum(dim=0).view(-1).cpu().numpy()
    assert np.allclose(q, (zq * zq).sum(axis=1), rtol=2e-3 if prec == S.PREC_BF16 else 1e-5)
    inside = (zq * zq).sum(axis=1) < wl.dml_margin
    assert inside[inp.labels == 0].any() and (~inside[inp.labels == 0]).any()      # both branches of the hinge
    for ctx, _ in shards:
        ctx.sfb_finish_factors(parts_all, G)
        ctx.sfb_gather_factors()
        ctx.sfb_apply_update()
        assert ctx.sfb_get_status() == 0
    Wsh = np.concatenate([w.cpu().numpy() for _, w in shards], axis=0)
    for ctx, _ in shards:
        ctx.close()
    err = rel_err(Wsh, ref, W0)
    print(f"dml {G} shards: rel err {err:.3e} (tol {TOL[prec]})")
    assert err <= TOL[prec]
    if G == 1:                                             # the helper on a single shard gives the same step
        W = to_dev(W0, torch)
        ctx = S.Context(S.make_config(S.DML, wl.rows, wl.cols, wl.workers, wl.batch, wl.eta, prec, dml_margin=wl.dml_margin), W)
        ctx.sfb_set_row_shard(0, wl.rows)
        part = torch.zeros((K, 1), dtype=torch.float32, device="cuda")
        sharded_step(ctx, X, lab, part, parts_all, torch.empty_like(X), torch.empty_like(lab), Y_local=Y, Y_all=torch.empty_like(Y))
        assert np.array_equal(W.cpu().numpy(), Wsh)
        ctx.close()
