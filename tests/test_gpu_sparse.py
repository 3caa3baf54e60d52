"""Sparse sufficient factors of MLR (Section 6: sparse features): samples in compressed-sparse-row form through
sfb_compute_factors_csr / sfb_step_csr against the oracle fed with the same samples as dense rows (zeros written out).
Every precision; the fused call and per-worker calls; a ragged shape (rows and columns not multiples of 32, odd and
empty columns); an entry-wise prox; the exchange-byte accounting; the dense update as the fallback when one worker
is dense; bad indices flagged and skipped."""
import numpy as np
import pytest

import paper_1409_5705_b200 as S
import sfb_inputs as I
from oracle import sfb_oracle as O
from _parity import TOL, rel_err, to_dev

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")

PRECS = [pytest.param(S.PREC_FP32_FFMA, id="ffma"), pytest.param(S.PREC_TF32X3, id="tf32x3"),
         pytest.param(S.PREC_BF16, id="bf16")]
WL = I.scaled(I.WORKLOADS["mlr_mid"], "mlr_sparse", rows=333, cols=268, workers=3, batch=37, eta=0.05, w_std=0.05,
              x_scale="unit")
WL_TILES = I.scaled(I.WORKLOADS["mlr_mid"], "mlr_sparse_tiles", rows=1000, cols=2052, workers=4, batch=64, eta=0.05,
                    w_std=0.05, x_scale="unit")


def _inputs(wl, step, nnz_mean):
    sp = I.sparse_samples(wl.seed, step, wl.K, wl.cols, nnz_mean)
    labels = I.zipf_labels(wl.seed, 5, step, wl.K, wl.rows, wl.zipf_s)
    return sp, labels


def _config(wl, prec, nnz_max, **kw):
    kw.setdefault("csr_update", S.CSR_UPDATE_SPARSE)        # these shapes are small: the cost model would go dense
    return S.make_config(wl.model, wl.rows, wl.cols, wl.workers, wl.batch, wl.eta, prec, csr_nnz_max=nnz_max, **kw)


def _entries_ok(Wg, ref, start, tol):
    """Entry-wise: within half an fp32 spacing of the oracle's value plus 8*tol of the entry's own update and of the rms
    update.  (With sparse samples the updates of the entries differ by orders of magnitude -- a popular column on a label
    row against a rare column elsewhere -- so the bound follows the entry; a missing or misplaced term is an error of the
    size of the entry's update and fails it.)"""
    upd = np.abs(ref - start)
    rms = float(np.sqrt((upd * upd).mean()))
    half_ulp = 0.5 * np.spacing(np.abs(ref).astype(np.float32)).astype(np.float64)
    return bool((np.abs(Wg.astype(np.float64) - ref) - half_ulp <= 8 * tol * (upd + rms)).all())


def _dev(sp, labels):
    return to_dev(sp.indptr, torch), to_dev(sp.indices, torch), to_dev(sp.values, torch), to_dev(labels, torch)


@pytest.mark.parametrize("prec", PRECS)
@pytest.mark.parametrize("wl", [pytest.param(WL, id="ragged"), pytest.param(WL_TILES, id="tiles")])
def test_sparse_steps_match_the_oracle_on_the_dense_form(wl, prec):
    W0 = I.initial_W(wl)
    W = to_dev(W0, torch)
    ctx = S.Context(_config(wl, prec, 40 * wl.K), W)
    start = W0.astype(np.float64)
    for step in range(2):
        sp, labels = _inputs(wl, step, 12.0)
        ip, ix, vl, lb = _dev(sp, labels)
        ctx.sfb_step_csr(ip, ix, vl, sp.nnz, lb)
        assert ctx.sfb_get_status() == 0
        Wg = W.cpu().numpy()
        # teacher-forced: the oracle steps from the W the GPU held before this step
        ref = O.sfb_step(I.MLR, start, I.densify(sp, wl.cols), None, labels, workers=wl.workers, eta=wl.eta)
        err = rel_err(Wg, ref, start)
        print(f"{wl.name} step {step}: err {err:.3e} (tol {TOL[prec]})")
        assert err <= TOL[prec]
        assert _entries_ok(Wg, ref, start, TOL[prec])
        start = Wg.astype(np.float64)
    st = ctx.sfb_get_stats()
    assert st.steps == 2
    if prec == S.PREC_BF16:
        # the bf16 operand copy follows the sparse update exactly
        copy = ctx.operand_copy_as_tensor()
        assert torch.equal(copy[:, :wl.cols].float(), W.to(torch.bfloat16).float())
    ctx.close()


@pytest.mark.parametrize("prec", [pytest.param(S.PREC_FP32_FFMA, id="ffma"), pytest.param(S.PREC_BF16, id="bf16")])
def test_per_worker_sparse_calls_equal_the_fused_call_bit_for_bit(prec):
    wl = WL
    W0 = I.initial_W(wl)
    sp, labels = _inputs(wl, 0, 9.0)
    out = []
    for fused in (True, False):
        W = to_dev(W0, torch)
        ctx = S.Context(_config(wl, prec, sp.nnz + 5), W)
        ip, ix, vl, lb = _dev(sp, labels)
        if fused:
            ctx.sfb_step_csr(ip, ix, vl, sp.nnz, lb)
        else:
            B = wl.batch
            for p in reversed(range(wl.workers)):       # any order of the workers
                n = int(sp.indptr[(p + 1) * B] - sp.indptr[p * B])
                ctx.sfb_compute_factors_csr(p, ip[p * B:], ix, vl, n, lb[p * B:])
            with pytest.raises(S.SfbError):              # a worker's triples are in the list once
                ctx.sfb_compute_factors_csr(0, ip, ix, vl, int(sp.indptr[B]), lb)
            ctx.sfb_gather_factors()
            ctx.sfb_apply_update()
        assert ctx.sfb_get_status() == 0
        out.append(W.cpu().numpy())
        ctx.close()
    assert np.array_equal(out[0], out[1])


def test_sparse_update_equals_the_dense_update_of_the_same_step():
    """One worker dense, the others sparse: the step takes the dense update; all sparse: the sparse one.  In fp32 both
    are the same sums up to their order."""
    wl = WL
    W0 = I.initial_W(wl)
    sp, labels = _inputs(wl, 0, 10.0)
    X = I.densify(sp, wl.cols)
    out, bytes_ = [], []
    for mixed in (False, True):
        W = to_dev(W0, torch)
        ctx = S.Context(_config(wl, S.PREC_FP32_FFMA, sp.nnz), W)
        ip, ix, vl, lb = _dev(sp, labels)
        B = wl.batch
        for p in range(wl.workers):
            if mixed and p == 1:
                ctx.sfb_compute_factors(p, to_dev(X[p * B:(p + 1) * B], torch), None, lb[p * B:])
            else:
                ctx.sfb_compute_factors_csr(p, ip[p * B:], ix, vl, int(sp.indptr[(p + 1) * B] - sp.indptr[p * B]), lb[p * B:])
        ctx.sfb_gather_factors()
        ctx.sfb_apply_update()
        assert ctx.sfb_get_status() == 0
        out.append(W.cpu().numpy().astype(np.float64))
        bytes_.append(ctx.sfb_get_stats().gather_bytes)
        ctx.close()
    upd = np.linalg.norm(out[0] - W0)
    assert np.linalg.norm(out[0] - out[1]) / upd < 1e-6
    # what the broadcast of the factors would move: u dense, v as (index, value) pairs when sparse
    assert bytes_[0] == wl.K * wl.rows * 4 + 8 * sp.nnz
    assert bytes_[1] == wl.K * (wl.rows + wl.cols) * 4


def test_sparse_step_with_l1_prox_matches_the_oracle():
    wl = WL
    W0 = I.initial_W(wl)
    sp, labels = _inputs(wl, 0, 12.0)
    W = to_dev(W0, torch)
    ctx = S.Context(_config(wl, S.PREC_FP32_FFMA, sp.nnz, prox_kind=S.PROX_L1, prox_weight=0.2), W)
    ctx.sfb_step_csr(*_dev(sp, labels)[:3], sp.nnz, to_dev(labels, torch))
    assert ctx.sfb_get_status() == 0
    Wg = W.cpu().numpy().astype(np.float64)
    ctx.close()
    X = I.densify(sp, wl.cols)
    ref = O.sfb_step(I.MLR, W0, X, None, labels, workers=wl.workers, eta=wl.eta, prox_kind="l1", prox_weight=0.2)
    plain = O.sfb_step(I.MLR, W0, X, None, labels, workers=wl.workers, eta=wl.eta)
    den = np.linalg.norm(plain - W0)
    assert np.linalg.norm(Wg - ref.astype(np.float32)) / den <= 1e-5 + np.linalg.norm(ref.astype(np.float32) - ref) / den
    assert (Wg[ref == 0.0] == 0.0).mean() > 0.999


def test_bad_indices_are_flagged_and_skipped_and_limits_are_errors():
    wl = WL
    W0 = I.initial_W(wl)
    sp, labels = _inputs(wl, 0, 8.0)
    bad = I.SparseSamples(sp.indptr.copy(), sp.indices.copy(), sp.values.copy())
    hit = [3, int(sp.indptr[50]) + 1]
    bad.indices[hit[0]] = wl.cols                        # out of range: entry skipped
    bad.indices[hit[1]] = -7
    W = to_dev(W0, torch)
    ctx = S.Context(_config(wl, S.PREC_FP32_FFMA, sp.nnz), W)
    ctx.sfb_step_csr(*_dev(bad, labels)[:3], sp.nnz, to_dev(labels, torch))
    assert ctx.sfb_get_status() == S.STATUS_INDEX_RANGE
    good = I.SparseSamples(sp.indptr, sp.indices.copy(), sp.values.copy())
    good.values[hit] = 0.0                               # the same samples without the two entries
    ref = O.sfb_step(I.MLR, W0, I.densify(good, wl.cols), None, labels, workers=wl.workers, eta=wl.eta)
    assert rel_err(W.cpu().numpy(), ref, W0) <= 1e-5
    # more entries than the context has room for; a context without room; a model without a sparse form
    with pytest.raises(S.SfbError) as e:
        ctx.sfb_step_csr(*_dev(sp, labels)[:3], sp.nnz + 1, to_dev(labels, torch))
    assert e.value.code == -3
    ctx.close()
    ctx = S.Context(_config(wl, S.PREC_FP32_FFMA, 0), to_dev(W0, torch))
    with pytest.raises(S.SfbError) as e:
        ctx.sfb_step_csr(*_dev(sp, labels)[:3], sp.nnz, to_dev(labels, torch))
    assert e.value.code == -10
    ctx.close()


@pytest.mark.parametrize("prec", [pytest.param(S.PREC_TF32X3, id="tf32x3"), pytest.param(S.PREC_BF16, id="bf16")])
def test_sparse_and_dense_steps_alternate_on_one_context(prec):
    """sparse, dense, sparse on the same context: no state of a sparse step leaks into the next step, and the operand
    copy of W that the forward products read stays current through both kinds of update."""
    wl = WL_TILES
    W0 = I.initial_W(wl)
    W = to_dev(W0, torch)
    ctx = S.Context(_config(wl, prec, 30 * wl.K), W)
    start = W0.astype(np.float64)
    for step, kind in enumerate(["sparse", "dense", "sparse"]):
        sp, labels = _inputs(wl, step, 10.0)
        X = I.densify(sp, wl.cols)
        if kind == "sparse":
            ctx.sfb_step_csr(*_dev(sp, labels)[:3], sp.nnz, to_dev(labels, torch))
        else:
            ctx.sfb_step(to_dev(X, torch), None, to_dev(labels, torch))
        assert ctx.sfb_get_status() == 0
        Wg = W.cpu().numpy()
        ref = O.sfb_step(I.MLR, start, X, None, labels, workers=wl.workers, eta=wl.eta)
        err = rel_err(Wg, ref, start)
        print(f"{kind} step {step}: err {err:.3e}")
        assert err <= TOL[prec]
        start = Wg.astype(np.float64)
    assert ctx.sfb_get_stats().sparse_updates == 2
    ctx.close()


def _manual_samples(rows_of_entries, cols):
    """CSR arrays from a list of per-sample [(column, value), ...] lists."""
    indptr = np.zeros(len(rows_of_entries) + 1, dtype=np.int64)
    idx, val = [], []
    for i, ents in enumerate(rows_of_entries):
        indptr[i + 1] = indptr[i] + len(ents)
        idx += [c for c, _ in ents]
        val += [v for _, v in ents]
    return I.SparseSamples(indptr, np.asarray(idx, dtype=np.int32), np.asarray(val, dtype=np.float32))


@pytest.mark.parametrize("prec", [pytest.param(S.PREC_FP32_FFMA, id="ffma"), pytest.param(S.PREC_BF16, id="bf16")])
def test_degenerate_sparse_batches(prec):
    """Empty samples, one sample with every column (more than one staging chunk of the row-wise forward and a column
    block longer than the update's entry window), columns no sample touches, unsorted indices, and a batch with no
    entry at all."""
    wl = I.scaled(I.WORKLOADS["mlr_mid"], "mlr_sparse_edge", rows=70, cols=300, workers=2, batch=5, eta=0.1, w_std=0.1,
                  x_scale="unit")
    rng = np.random.default_rng(3)
    full = [(int(c), float(v)) for c, v in zip(rng.permutation(wl.cols), rng.standard_normal(wl.cols) * 0.1)]
    few = [(299, 0.5), (0, -0.25), (17, 1.0)]                                  # unsorted, first and last column
    samples = [[], full, few, [], [(5, 2.0)], full[:200], [], [(5, -1.0), (6, 1.0)], few[::-1], []]
    sp = _manual_samples(samples, wl.cols)
    labels = I.zipf_labels(wl.seed, 5, 0, wl.K, wl.rows, 0.0)
    W0 = I.initial_W(wl)
    W = to_dev(W0, torch)
    ctx = S.Context(_config(wl, prec, sp.nnz + 8), W)
    ctx.sfb_step_csr(*_dev(sp, labels)[:3], sp.nnz, to_dev(labels, torch))
    assert ctx.sfb_get_status() == 0
    ref = O.sfb_step(I.MLR, W0, I.densify(sp, wl.cols), None, labels, workers=wl.workers, eta=wl.eta)
    assert rel_err(W.cpu().numpy(), ref, W0) <= TOL[prec]
    # a batch without a single entry: u = softmax(0) - onehot, v = 0, W unchanged
    before = W.clone()
    empty = _manual_samples([[] for _ in range(wl.K)], wl.cols)
    ip = to_dev(empty.indptr, torch)
    dummy_i = torch.zeros(1, dtype=torch.int32, device="cuda")
    dummy_v = torch.zeros(1, dtype=torch.float32, device="cuda")
    ctx.sfb_step_csr(ip, dummy_i, dummy_v, 0, to_dev(labels, torch))
    assert ctx.sfb_get_status() == 0
    assert torch.equal(W, before)
    assert ctx.sfb_get_stats().sparse_updates == 2
    ctx.close()


def test_a_batch_too_large_for_the_factor_slab_takes_the_dense_update():
    wl = I.scaled(I.WORKLOADS["mlr_mid"], "mlr_sparse_bigk", rows=64, cols=64, workers=4, batch=640, eta=0.05, w_std=0.1,
                  x_scale="unit")                                                 # K = 2560: beyond the slab in either mode
    sp, labels = _inputs(wl, 0, 4.0)
    W0 = I.initial_W(wl)
    W = to_dev(W0, torch)
    ctx = S.Context(_config(wl, S.PREC_FP32_FFMA, sp.nnz), W)
    ctx.sfb_step_csr(*_dev(sp, labels)[:3], sp.nnz, to_dev(labels, torch))
    assert ctx.sfb_get_status() == 0
    assert ctx.sfb_get_stats().sparse_updates == 0
    ref = O.sfb_step(I.MLR, W0, I.densify(sp, wl.cols), None, labels, workers=wl.workers, eta=wl.eta)
    assert rel_err(W.cpu().numpy(), ref, W0) <= 1e-5
    ctx.close()
