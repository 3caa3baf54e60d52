"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle on the same seeded inputs."""
import numpy as np
import pytest

import paper_1409_5705_b200 as S
import sfb_inputs as I
from oracle import sfb_oracle as O
from _parity import TOL, step_tol, config_for, oracle_step, rel_err, to_dev

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")

PRECS = [pytest.param(S.PREC_FP32, id="fp32"), pytest.param(S.PREC_BF16, id="bf16")]


def small(name):
    """Ragged shapes spanning several 128-wide tiles with tails, same recipes as the full workloads."""
    if name == "mlr":
        return I.scaled(I.WORKLOADS["mlr_mid"], "mlr_small", rows=333, cols=260, workers=3, batch=37, eta=0.05,
                        w_std=0.05, x_scale="unit")
    if name == "dml":
        return I.scaled(I.WORKLOADS["dml"], "dml_small", rows=150, cols=388, workers=4, batch=33, eta=1e-3)
    if name == "sc":
        return I.scaled(I.WORKLOADS["sc"], "sc_small", rows=300, cols=200, workers=3, batch=11, eta=1e-2,
                        sc_nnz=6)
    raise KeyError(name)


def gpu_step(wl, W0, inp, prec, L=0.0, per_worker=False, dense=False):
    W = to_dev(W0, torch)
    ctx = S.Context(config_for(wl, prec, L), W)
    X, Y, lab = to_dev(inp.X, torch), to_dev(inp.Y, torch), to_dev(inp.labels, torch)
    if dense:
        scratch = torch.empty(2 * wl.rows * wl.cols, dtype=torch.float32, device="cuda")
        ctx.sfb_dense_sync_step(X, Y, lab, scratch)
    elif per_worker:
        B = wl.batch
        for p in reversed(range(wl.workers)):            # any order: each worker owns its rows
            ctx.sfb_compute_factors(p, X[p * B:(p + 1) * B], None if Y is None else Y[p * B:(p + 1) * B],
                                    None if lab is None else lab[p * B:(p + 1) * B])
        ctx.sfb_gather_factors()
        ctx.sfb_apply_update()
    else:
        ctx.sfb_step(X, Y, lab)
    U, V = ctx.factors_as_tensors()
    st = ctx.sfb_get_status()
    stats = ctx.sfb_get_stats()
    out = W.cpu().numpy(), U.cpu().numpy(), V.cpu().numpy(), st, stats
    ctx.close()
    return out


@pytest.mark.parametrize("prec", PRECS)
def test_mlr_tiny_all_steps_teacher_forced(prec):
    """MLR tiny, all 16 steps; each step is compared from the GPU's own W_t (single steps are what is pinned)."""
    wl = I.WORKLOADS["mlr_tiny"]
    W = to_dev(I.initial_W(wl), torch)
    ctx = S.Context(config_for(wl, prec), W)
    for t in range(wl.steps):
        inp = I.step_inputs(wl, t)
        Wt = W.cpu().numpy()
        ctx.sfb_step(to_dev(inp.X, torch), None, to_dev(inp.labels, torch))
        ref = oracle_step(wl, Wt, inp)
        assert rel_err(W.cpu().numpy(), ref, Wt) <= TOL[prec], f"step {t}"
        if t == 0:   # zero-init: p = 1/64 exactly, the loss is log 64
            assert abs(ctx.sfb_get_stats().last_loss - np.log(64.0)) < 1e-5
    assert ctx.sfb_get_status() == 0
    st = ctx.sfb_get_stats()
    assert st.steps == wl.steps and st.samples == wl.steps * wl.K
    ctx.close()


@pytest.mark.parametrize("prec", PRECS)
@pytest.mark.parametrize("name", ["mlr", "dml", "sc"])
def test_small_ragged_step_matches_oracle(name, prec):
    wl = small(name)
    W0 = I.initial_W(wl)
    if name == "dml":
        W0 = (W0 * np.float32(0.06)).astype(np.float32)          # puts dissimilar pairs on both sides of the margin
    inp = I.step_inputs(wl, 0)
    L = O.lipschitz_power_iteration(W0) if name == "sc" else 0.0
    Wref, Uref, Vref = oracle_step(wl, W0, inp, L=L, return_factors=True)
    if name == "dml":
        q = ((Vref @ W0.astype(np.float64).T) ** 2).sum(axis=1)
        dis = inp.labels == 0
        assert (q[dis] < 1).any() and (q[dis] >= 1).any()       # both hinge branches are exercised
        assert O.dml_hinge_distance(W0, inp.X, inp.Y, inp.labels) > 4e-3   # no pair sits on the kink
    Wg, Ug, Vg, status, stats = gpu_step(wl, W0, inp, prec, L)
    assert status == 0
    assert rel_err(Wg, Wref, W0) <= step_tol(wl, prec, Wref, W0)
    ftol = 1e-5 if prec == S.PREC_FP32 else 1e-2
    if name == "mlr" and prec == S.PREC_BF16:
        # bf16 mode leaves the label entry u_iy = p_iy - 1 out of the bf16 operand (it holds 0 there) and applies
        # it to W in fp32: the operand must be exactly 0 at (i, y_i); the rest is compared with the oracle's u
        assert (Ug[np.arange(wl.K), inp.labels] == 0).all()
        Ug[np.arange(wl.K), inp.labels] = Uref[np.arange(wl.K), inp.labels]
    assert np.linalg.norm(Ug - Uref) <= ftol * np.linalg.norm(Uref)
    assert np.linalg.norm(Vg - Vref) <= ftol * max(np.linalg.norm(Vref), 1e-30)
    if name == "mlr":
        # integer handling is exact: the one entry of u_i below zero sits at the class id
        np.testing.assert_array_equal(Ug.argmin(axis=1), inp.labels)
        assert abs(stats.last_loss - O.mlr_loss(W0, inp.X, inp.labels).mean()) < 1e-4
    if name == "dml":
        zero_rows = np.abs(Uref).sum(axis=1) == 0
        assert zero_rows.any()
        assert (np.abs(Ug[zero_rows]).sum(axis=1) == 0).all()   # inactive hinge: u is exactly 0
    if name == "sc":
        norms = np.linalg.norm(Wg.astype(np.float64), axis=0)
        assert (norms <= 1 + 1e-6).all()
        assert abs(stats.sc_lipschitz - L) <= 1e-6 * L
    # the byte report of the cost table
    esz = 2 if (prec == S.PREC_BF16 and name == "mlr") else 4     # DML, SC: fp32 or a (hi, lo) bf16 pair
    one, p2p, fms = O.comm_values(wl.rows, wl.cols, wl.workers, wl.batch)
    assert stats.gather_bytes == one * esz and stats.gather_bytes_p2p == p2p * esz
    assert stats.dense_sync_bytes == fms * 4


@pytest.mark.parametrize("prec", PRECS)
@pytest.mark.parametrize("name", ["mlr", "dml", "sc"])
def test_three_steps_teacher_forced_on_ragged_shapes(name, prec):
    """Several steps on one context: whatever the library keeps between steps (the bf16 copy of W and its label
    rows, the split copies of W rebuilt at the start of a step) must follow W.  Each step is compared with one
    oracle step from the GPU's own W_t."""
    wl = small(name)
    W0 = I.initial_W(wl)
    if name == "dml":
        W0 = (W0 * np.float32(0.06)).astype(np.float32)
    W = to_dev(W0, torch)
    L0 = O.lipschitz_power_iteration(W0) if name == "sc" else 0.0
    ctx = S.Context(config_for(wl, prec, L0 * 1.05), W)       # any step 1/L with L >= ||W||^2 is a valid ISTA step
    true_dict = I.sc_true_dictionary(wl) if name == "sc" else None
    for t in range(3):
        inp = I.step_inputs(wl, t, true_dict)
        Wt = W.cpu().numpy()
        if name == "dml" and O.dml_hinge_distance(Wt, inp.X, inp.Y, inp.labels) < 4e-3:
            continue                                           # a pair on the kink: two answers are correct
        ctx.sfb_step(to_dev(inp.X, torch), to_dev(inp.Y, torch), to_dev(inp.labels, torch))
        ref = oracle_step(wl, Wt, inp, L=float(np.float32(L0 * 1.05)) if name == "sc" else None)
        assert rel_err(W.cpu().numpy(), ref, Wt) <= step_tol(wl, prec, ref, Wt), f"step {t}"
    assert ctx.sfb_get_status() == 0
    ctx.close()


@pytest.mark.parametrize("prec", PRECS)
@pytest.mark.parametrize("name", ["mlr", "dml", "sc"])
def test_per_worker_calls_equal_the_fused_step(name, prec):
    """P calls of sfb_compute_factors (any order) + gather + apply == sfb_step: BSP, same W for all workers."""
    wl = small(name)
    W0, inp = I.initial_W(wl), I.step_inputs(wl, 1)
    if name == "dml":
        W0 = (W0 * np.float32(0.06)).astype(np.float32)
    L = O.lipschitz_power_iteration(W0) if name == "sc" else 0.0
    Wa = gpu_step(wl, W0, inp, prec, L)[0]
    Wb = gpu_step(wl, W0, inp, prec, L, per_worker=True)[0]
    ref = oracle_step(wl, W0, inp, L=L)
    tol = step_tol(wl, prec, ref, W0)
    assert rel_err(Wb, ref, W0) <= tol
    if prec == S.PREC_FP32:
        np.testing.assert_array_equal(Wa, Wb)
    else:
        assert rel_err(Wb, Wa.astype(np.float64), W0) <= tol


def test_worker_split_invariance_and_determinism():
    """(P=4, B=32) and (P=1, B=128) give the same W; repeated runs are bit-identical (BSP, Section 4.1)."""
    wl4 = I.WORKLOADS["mlr_tiny"]
    wl1 = I.scaled(wl4, "one_worker", workers=1, batch=128)
    W0 = I.normal_matrix(0, 9, wl4.rows, wl4.cols, 0.1)
    inp = I.step_inputs(wl4, 3)
    a = gpu_step(wl4, W0, inp, S.PREC_FP32)[0]
    b = gpu_step(wl1, W0, inp, S.PREC_FP32)[0]
    c = gpu_step(wl4, W0, inp, S.PREC_FP32)[0]
    np.testing.assert_array_equal(a, b)
    np.testing.assert_array_equal(a, c)


@pytest.mark.parametrize("name", ["mlr", "dml", "sc"])
def test_dense_sync_path_makes_the_same_progress(name):
    """Full-matrix synchronisation and SFB produce the same W per step (Experiments, progress per sample)."""
    wl = small(name)
    W0, inp = I.initial_W(wl), I.step_inputs(wl, 2)
    L = O.lipschitz_power_iteration(W0) if name == "sc" else 0.0
    ref = oracle_step(wl, W0, inp, L=L)
    Wd = gpu_step(wl, W0, inp, S.PREC_FP32, L, dense=True)[0]
    Ws = gpu_step(wl, W0, inp, S.PREC_FP32, L)[0]
    assert rel_err(Wd, ref, W0) <= step_tol(wl, S.PREC_FP32, ref, W0)
    assert rel_err(Wd, Ws.astype(np.float64), W0) <= step_tol(wl, S.PREC_FP32, ref, W0)


def test_library_lipschitz_estimate_matches_power_iteration():
    wl = small("sc")
    W0, inp = I.initial_W(wl), I.step_inputs(wl, 0)
    Lref = O.lipschitz_power_iteration(W0, 50)
    Wg, _, _, _, stats = gpu_step(wl, W0, inp, S.PREC_FP32, L=0.0)
    assert abs(stats.sc_lipschitz - Lref) <= 1e-5 * Lref
    ref = oracle_step(wl, W0, inp, L=float(np.float32(stats.sc_lipschitz)))
    assert rel_err(Wg, ref, W0) <= step_tol(wl, S.PREC_FP32, ref, W0)


def test_call_order_and_label_range_are_reported_not_trapped():
    wl = small("mlr")
    W0, inp = I.initial_W(wl), I.step_inputs(wl, 0)
    W = to_dev(W0, torch)
    ctx = S.Context(config_for(wl, S.PREC_FP32), W)
    X, lab = to_dev(inp.X, torch), to_dev(inp.labels, torch)
    with pytest.raises(S.SfbError) as e:
        ctx.sfb_gather_factors()
    assert e.value.code == -9
    ctx.sfb_compute_factors(0, X[:wl.batch], None, lab[:wl.batch])
    with pytest.raises(S.SfbError) as e:
        ctx.sfb_gather_factors()                       # workers 1, 2 have not committed
    assert e.value.code == -9
    with pytest.raises(S.SfbError) as e:
        ctx.sfb_apply_update()
    assert e.value.code == -9
    with pytest.raises(S.SfbError) as e:
        ctx.sfb_compute_factors(wl.workers, X, None, lab)
    assert e.value.code == -3
    bad = inp.labels.copy()
    bad[5] = wl.rows
    bad[7] = -1
    ctx.sfb_step(X, None, to_dev(bad, torch))
    assert ctx.sfb_get_status() == S.STATUS_LABEL_RANGE
    assert ctx.sfb_get_status() == 0                   # reading clears it
    U, _ = ctx.factors_as_tensors()
    U = U.cpu().numpy()
    assert abs(U[5].sum() - 1.0) < 1e-4 and abs(U[7].sum() - 1.0) < 1e-4 and abs(U[6].sum()) < 1e-4
    ctx.close()


def test_host_buffer_step_matches_device_step():
    wl = small("mlr")
    W0, inp = I.initial_W(wl), I.step_inputs(wl, 4)
    Wa = gpu_step(wl, W0, inp, S.PREC_FP32)[0]
    W = to_dev(W0, torch)
    ctx = S.Context(config_for(wl, S.PREC_FP32), W)
    Xh = torch.from_numpy(inp.X).pin_memory()
    yh = torch.from_numpy(inp.labels).pin_memory()
    loss, status = ctx.sfb_step_host(Xh, None, yh)
    assert status == 0 and abs(loss - O.mlr_loss(W0, inp.X, inp.labels).mean()) < 1e-4
    np.testing.assert_array_equal(W.cpu().numpy(), Wa)
    ctx.close()


@pytest.mark.parametrize("prec", PRECS)
@pytest.mark.parametrize("name", ["dml", "sc"])
def test_host_buffer_step_for_pairs_and_codes(name, prec):
    """sfb_step_host stages X (and the pair partner and the flags) itself: same W as the device-resident step."""
    wl = small(name)
    W0 = I.initial_W(wl)
    if name == "dml":
        W0 = (W0 * np.float32(0.06)).astype(np.float32)
    inp = I.step_inputs(wl, 5, I.sc_true_dictionary(wl) if name == "sc" else None)
    L = O.lipschitz_power_iteration(W0) if name == "sc" else 0.0
    Wa = gpu_step(wl, W0, inp, prec, L)[0]
    W = to_dev(W0, torch)
    ctx = S.Context(config_for(wl, prec, L), W)
    pin = lambda a: None if a is None else torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    loss, status = ctx.sfb_step_host(pin(inp.X), pin(inp.Y), pin(inp.labels))
    assert status == 0 and loss == 0.0
    np.testing.assert_array_equal(W.cpu().numpy(), Wa)
    ctx.close()


def test_two_contexts_on_two_streams_step_concurrently():
    """One context per stream: two independent problems stepped from two streams at once (their kernels all want
    the whole tensor memory and most of the shared memory of an SM, so they take turns) both match the oracle."""
    wl = small("mlr")
    ctxs = []
    for k in range(2):
        W0, inp = I.initial_W(wl), I.step_inputs(wl, 10 + k)
        W0 = (W0 * np.float32(1.0 + 0.5 * k)).astype(np.float32)
        stream = torch.cuda.Stream()
        W = to_dev(W0, torch)
        X, lab = to_dev(inp.X, torch), to_dev(inp.labels, torch)
        torch.cuda.synchronize()
        ctx = S.Context(config_for(wl, S.PREC_BF16), W, stream=stream)
        ctxs.append((ctx, W, W0, inp, X, lab))
    for ctx, W, W0, inp, X, lab in ctxs:                 # interleave the launches of the two streams
        ctx.sfb_compute_factors(-1, X, None, lab)
    for ctx, *_ in ctxs:
        ctx.sfb_gather_factors()
    for ctx, *_ in ctxs:
        ctx.sfb_apply_update()
    torch.cuda.synchronize()
    for ctx, W, W0, inp, X, lab in ctxs:
        assert ctx.sfb_get_status() == 0
        ref = oracle_step(wl, W0, inp)
        assert rel_err(W.cpu().numpy(), ref, W0) <= TOL[S.PREC_BF16]
        ctx.close()
