"""Seeded input generators: determinism, block independence, label ranges and the stated distributions."""
import numpy as np

import sfb_inputs as I


def test_blocks_are_independent_of_the_split():
    a = I.normal_matrix(0, 1, 9000, 16, 0.01, threads=4)
    b = I.normal_matrix(0, 1, 9000, 16, 0.01, threads=1)
    c = I.normal_rows(0, 1, 4096, 9000, 16, 0.01)
    np.testing.assert_array_equal(a, b)
    np.testing.assert_array_equal(a[4096:], c)
    assert a.dtype == np.float32 and abs(a.std() - 0.01) < 2e-4


def test_step_inputs_are_deterministic_and_in_range():
    for name in ("mlr_tiny",):
        wl = I.WORKLOADS[name]
        s0, s0b, s1 = I.step_inputs(wl, 0), I.step_inputs(wl, 0), I.step_inputs(wl, 1)
        np.testing.assert_array_equal(s0.X, s0b.X)
        np.testing.assert_array_equal(s0.labels, s0b.labels)
        assert not np.array_equal(s0.X, s1.X)
        assert s0.X.shape == (wl.K, wl.cols) and s0.labels.dtype == np.int32
        assert s0.labels.min() >= 0 and s0.labels.max() < wl.rows
    assert (I.initial_W(I.WORKLOADS["mlr_tiny"]) == 0).all()


def test_zipf_labels_follow_the_power_law():
    y = I.zipf_labels(0, 5, 0, 200_000, 1000, 1.1)
    assert y.min() >= 0 and y.max() < 1000
    c = np.bincount(y, minlength=1000).astype(np.float64)
    w = np.arange(1, 1001) ** -1.1
    w /= w.sum()
    assert abs(c[0] / c.sum() - w[0]) < 0.01 and abs(c[9] / c.sum() - w[9]) < 0.005


def test_small_dml_and_sc_recipes():
    wl = I.scaled(I.WORKLOADS["dml"], "dml_small", rows=12, cols=40, workers=2, batch=8)
    s = I.step_inputs(wl, 3)
    sim = s.labels == 1
    assert set(np.unique(s.labels)) <= {0, 1}
    d = np.linalg.norm(s.X - s.Y, axis=1)
    assert (d[sim] < 0.1 * np.sqrt(40) * 2).all() and (d[~sim] > 3).all()
    wl = I.scaled(I.WORKLOADS["sc"], "sc_small", rows=64, cols=48, workers=2, batch=4, sc_nnz=5)
    W0 = I.initial_W(wl)
    np.testing.assert_allclose(np.linalg.norm(W0.astype(np.float64), axis=0), 1.0, atol=1e-6)
    s = I.step_inputs(wl, 0)
    assert s.X.shape == (8, 64) and s.Y is None and s.labels is None
