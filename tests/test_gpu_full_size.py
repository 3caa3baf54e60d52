"""Parity at the full sizes of the five workloads, one step each, in the launch configuration the bench times.
The paper-scale MLR shape is checked on sampled rows of W (every label row, random rows, the last rows),
which the oracle computes from the exact log-partition of every sample."""
import numpy as np
import pytest

import paper_1409_5705_b200 as S
import sfb_inputs as I
from oracle import sfb_oracle as O
from _parity import (TOL, step_tol, config_for, entries_excess, entries_ok, oracle_step, rel_err, storage_floor,
                     to_dev)

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")

PRECS = [pytest.param(S.PREC_FP32, id="fp32"), pytest.param(S.PREC_BF16, id="bf16")]


@pytest.mark.parametrize("prec", PRECS)
@pytest.mark.parametrize("name", ["mlr_mid", "dml", "sc"])
def test_full_size_step(name, prec):
    wl = I.WORKLOADS[name]
    W0 = I.initial_W(wl)
    inp = I.step_inputs(wl, 0)
    L = float(np.float32(O.lipschitz_power_iteration(W0))) if wl.model == I.SC else 0.0
    W = to_dev(W0, torch)
    ctx = S.Context(config_for(wl, prec, L), W)
    ctx.sfb_step(to_dev(inp.X, torch), to_dev(inp.Y, torch), to_dev(inp.labels, torch))
    assert ctx.sfb_get_status() == 0
    Wg = W.cpu().numpy()
    ctx.close()
    del W
    torch.cuda.empty_cache()
    ref = oracle_step(wl, W0, inp, L=L)
    err = rel_err(Wg, ref, W0)
    tol = step_tol(wl, prec, ref, W0)
    stores = 2 if wl.model == I.SC else 1                       # sparse coding stores W twice (update, then prox)
    print(f"{name}: rel err {err:.3e}, tolerance {tol:.3e} (stated {TOL[prec]:.0e} + storage floor "
          f"{storage_floor(ref, W0):.2e} x {stores if wl.model == I.SC else 0}); worst entry beyond its storage "
          f"rounding {entries_excess(Wg, ref, W0, stores):.3e} rms updates (allowed {8 * TOL[prec]:.1e})")
    assert err <= tol, err
    # rows that carry no label and the ragged last tile must be right on their own, not hidden by the norm
    tail = slice(wl.rows - wl.rows % 128 if wl.rows % 128 else wl.rows - 128, wl.rows)
    if wl.model != I.MLR:
        assert rel_err(Wg[tail], ref[tail], W0[tail]) <= 2 * tol
        assert entries_ok(Wg, ref, W0, TOL[prec], stores)       # every entry of the matrix, not only its norm
        assert entries_ok(Wg[tail], ref[tail], W0[tail], TOL[prec], stores)
    else:
        assert entries_ok(Wg[tail], ref[tail], W0[tail], TOL[prec])
        bulk = np.setdiff1d(np.arange(wl.rows), inp.labels)
        assert entries_ok(Wg[bulk], ref[bulk], W0[bulk], TOL[prec])


def test_sparse_coding_without_prox_meets_the_bound_plus_one_storage_floor():
    """fp32 operands, no prox: W is stored once, so the error against the once-rounded oracle may exceed 1e-5 by at
    most one storage floor (with the prox it is two)."""
    wl = I.WORKLOADS["sc"]
    W0 = I.initial_W(wl)
    inp = I.step_inputs(wl, 0, I.sc_true_dictionary(wl))
    L = float(np.float32(O.lipschitz_power_iteration(W0)))
    W = to_dev(W0, torch)
    ctx = S.Context(config_for(wl, S.PREC_FP32, L, prox=0), W)
    ctx.sfb_step(to_dev(inp.X, torch), None, None)
    assert ctx.sfb_get_status() == 0
    Wg = W.cpu().numpy()
    ctx.close()
    ref = O.sfb_step(wl.model, W0, inp.X, None, None, workers=wl.workers, eta=wl.eta, lam=wl.sc_lambda, L=L,
                     iters=wl.sc_iters, prox=False)
    err, floor = rel_err(Wg, ref, W0), storage_floor(ref, W0)
    print(f"sc without prox: rel err {err:.3e}, storage floor {floor:.3e}")
    assert err <= TOL[S.PREC_FP32] + floor
    assert entries_ok(Wg, ref, W0, TOL[S.PREC_FP32])


def test_mlr_large_three_steps_teacher_forced_on_sampled_rows():
    """bf16 mode at the paper-scale shape, three steps: steps 2 and 3 run their forward product on the bf16 copy of W
    that the update of the step before wrote (label rows and the ragged last tile included), so they verify that copy
    at the size where it matters.  Each step is checked from the GPU's own W_t on sampled rows."""
    wl = I.WORKLOADS["mlr_large"]
    W0 = I.initial_W(wl, threads=16)
    W = torch.empty((wl.rows, wl.cols), dtype=torch.float32, device="cuda")
    chunk = 32768
    for r0 in range(0, wl.rows, chunk):
        W[r0:r0 + chunk].copy_(torch.from_numpy(W0[r0:r0 + chunk]))
    ctx = S.Context(config_for(wl, S.PREC_BF16), W)
    Wt = W0                                                     # host copy of the W the step starts from
    rng = np.random.default_rng(11)
    for t in range(3):
        inp = I.step_inputs(wl, t)
        ctx.sfb_step(to_dev(inp.X, torch), None, to_dev(inp.labels, torch))
        assert ctx.sfb_get_status() == 0
        label_rows = np.unique(inp.labels)
        rows = np.unique(np.concatenate([label_rows, rng.integers(0, wl.rows, 2048),
                                         np.arange(wl.rows - 136, wl.rows)]))
        Wg = W[torch.from_numpy(rows).cuda()].cpu().numpy()
        lse = O.mlr_log_partition(Wt, inp.X)
        ref = O.mlr_updated_rows(Wt[rows], rows, inp.X, inp.labels, lse, wl.eta)
        W0r = Wt[rows]
        err = rel_err(Wg, ref, W0r)
        print(f"mlr_large step {t}: rel err on {len(rows)} sampled rows {err:.3e}")
        assert err <= TOL[S.PREC_BF16], (t, err)
        is_label = np.isin(rows, label_rows)
        assert entries_ok(Wg[~is_label], ref[~is_label], W0r[~is_label], TOL[S.PREC_BF16]), t
        if t < 2:                                               # the next step starts from what the GPU holds now
            Wt = np.empty_like(W0)
            for r0 in range(0, wl.rows, chunk):
                Wt[r0:r0 + chunk] = W[r0:r0 + chunk].cpu().numpy()
    ctx.close()
    del W
    torch.cuda.empty_cache()


@pytest.mark.parametrize("prec", PRECS)
def test_mlr_large_sampled_rows(prec):
    wl = I.WORKLOADS["mlr_large"]
    W0 = I.initial_W(wl, threads=16)
    inp = I.step_inputs(wl, 0)
    W = torch.empty((wl.rows, wl.cols), dtype=torch.float32, device="cuda")
    chunk = 32768
    for r0 in range(0, wl.rows, chunk):
        W[r0:r0 + chunk].copy_(torch.from_numpy(W0[r0:r0 + chunk]))
    ctx = S.Context(config_for(wl, prec), W)
    ctx.sfb_step(to_dev(inp.X, torch), None, to_dev(inp.labels, torch))
    assert ctx.sfb_get_status() == 0
    loss = ctx.sfb_get_stats().last_loss
    rng = np.random.default_rng(7)
    label_rows = np.unique(inp.labels)
    rows = np.unique(np.concatenate([label_rows, rng.integers(0, wl.rows, 4096),
                                     np.arange(wl.rows - 136, wl.rows)]))
    Wg = W[torch.from_numpy(rows).cuda()].cpu().numpy()
    ctx.close()
    del W
    torch.cuda.empty_cache()
    lse = O.mlr_log_partition(W0, inp.X)
    ref = O.mlr_updated_rows(W0[rows], rows, inp.X, inp.labels, lse, wl.eta)
    W0r = W0[rows]
    assert rel_err(Wg, ref, W0r) <= TOL[prec]
    is_label = np.isin(rows, label_rows)
    assert entries_ok(Wg[~is_label], ref[~is_label], W0r[~is_label], TOL[prec])
    last = rows >= wl.rows - 136
    assert entries_ok(Wg[last], ref[last], W0r[last], TOL[prec])
    zy = np.einsum("kd,kd->k", inp.X.astype(np.float64), W0[inp.labels].astype(np.float64))
    assert abs(loss - float((lse - zy).mean())) < 1e-3


@pytest.mark.parametrize("prec", PRECS)
def test_mlr_large_sparse_samples_sampled_rows(prec):
    """The paper-scale shape with sparse samples (about 100 non-zeros each) through the sparse update, against the
    oracle on the same samples written out densely."""
    wl = I.WORKLOADS["mlr_large"]
    W0 = I.initial_W(wl, threads=16)
    labels = I.step_inputs(wl, 0).labels
    sp = I.sparse_samples(wl.seed, 0, wl.K, wl.cols, 100.0)
    X = I.densify(sp, wl.cols)
    W = torch.empty((wl.rows, wl.cols), dtype=torch.float32, device="cuda")
    chunk = 32768
    for r0 in range(0, wl.rows, chunk):
        W[r0:r0 + chunk].copy_(torch.from_numpy(W0[r0:r0 + chunk]))
    cfg = S.make_config(wl.model, wl.rows, wl.cols, wl.workers, wl.batch, wl.eta, prec, csr_nnz_max=sp.nnz,
                        csr_update=S.CSR_UPDATE_SPARSE)
    ctx = S.Context(cfg, W)
    ctx.sfb_step_csr(to_dev(sp.indptr, torch), to_dev(sp.indices, torch), to_dev(sp.values, torch), sp.nnz,
                     to_dev(labels, torch))
    assert ctx.sfb_get_status() == 0
    st = ctx.sfb_get_stats()
    assert st.sparse_updates == 1
    rng = np.random.default_rng(11)
    label_rows = np.unique(labels)
    rows = np.unique(np.concatenate([label_rows, rng.integers(0, wl.rows, 4096), np.arange(wl.rows - 136, wl.rows)]))
    Wg = W[torch.from_numpy(rows).cuda()].cpu().numpy()
    if prec == S.PREC_BF16:                      # the operand copy follows the sparse update exactly
        copy = ctx.operand_copy_as_tensor()
        sel = torch.from_numpy(rows[::16]).cuda()
        assert torch.equal(copy[sel][:, :wl.cols].float(), W[sel].to(torch.bfloat16).float())
    ctx.close()
    del W
    torch.cuda.empty_cache()
    lse = O.mlr_log_partition(W0, X)
    ref = O.mlr_updated_rows(W0[rows], rows, X, labels, lse, wl.eta)
    W0r = W0[rows]
    err = rel_err(Wg, ref, W0r)
    print(f"mlr_large sparse: rel err on {len(rows)} rows {err:.3e} (tol {TOL[prec]})")
    assert err <= TOL[prec]
    # entry-wise, the bound following the entry's own update (updates of sparse samples span orders of magnitude)
    upd = np.abs(ref - W0r)
    rms = float(np.sqrt((upd * upd).mean()))
    half_ulp = 0.5 * np.spacing(np.abs(ref).astype(np.float32)).astype(np.float64)
    is_label = np.isin(rows, label_rows)
    ok = np.abs(Wg.astype(np.float64) - ref) - half_ulp <= 8 * TOL[prec] * (upd + rms)
    assert ok[~is_label].all()
    assert abs(st.last_loss - float((lse - np.einsum("kd,kd->k", X.astype(np.float64),
                                                      W0[labels].astype(np.float64))).mean())) < 1e-3
