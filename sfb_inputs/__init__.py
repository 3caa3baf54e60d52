"""Seeded synthetic inputs for the SFB hot path (shared by the tests, the bench and the smoke check).

This module only *draws inputs*: parameter matrices, samples, labels, similarity flags.  It contains none
of the method's arithmetic (no sufficient factors, no softmax, no ISTA, no update), so that the CPU oracle and
the CUDA path can both be fed from it without sharing any of the computation under test.

Generator: numpy's counter-based Philox, keyed by ``(seed, stream, block)``.  Every array is produced in
independent row blocks, so a block can be regenerated alone (the 13 GB matrix of the paper-scale MLR shape is
drawn block by block, in threads) and the values do not depend on the block-parallel schedule.

The five workloads mirror the shapes of the paper's experiments (Section "Experiments": 325k classes,
10k-20k features, billions of matrix entries) with dense synthetic features standing in for its datasets.
"""
from __future__ import annotations

import math
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field

import numpy as np

MLR, DML, SC = 0, 1, 2

# stream ids
_S_W0, _S_WTRUE, _S_X, _S_Y, _S_LABEL, _S_SUPPORT, _S_NOISE, _S_CODEVAL = 1, 2, 3, 4, 5, 6, 7, 8

_BLOCK_ROWS = 4096


@dataclass(frozen=True)
class Workload:
    """One synthetic workload: shape of W, logical workers, step count and the input recipe."""
    name: str
    model: int
    rows: int            # MLR: classes J | DML: latent dim k | SC: feature dim D
    cols: int            # MLR/DML: feature dim D | SC: atoms A
    workers: int         # P
    batch: int           # B ; K = P*B pairs per step
    eta: float
    steps: int
    seed: int = 0
    w_init: str = "normal"       # "zeros" | "normal" | "dml" | "unit_columns"
    w_std: float = 0.01
    zipf_s: float = 0.0          # 0 -> uniform labels
    x_scale: str = "unit"        # "unit" | "inv_sqrt_d"
    n_samples: int = 0           # >0: a fixed pool swept deterministically (MLR tiny)
    sc_lambda: float = 0.1
    sc_iters: int = 20
    sc_nnz: int = 20
    sc_noise: float = 0.01
    dml_margin: float = 1.0
    dml_pair_noise: float = 0.1
    extra: dict = field(default_factory=dict)

    @property
    def K(self) -> int:
        return self.workers * self.batch

    @property
    def in_dim(self) -> int:
        """Length of one input sample x: the feature dimension."""
        return self.rows if self.model == SC else self.cols


WORKLOADS = {
    "mlr_tiny": Workload("mlr_tiny", MLR, 64, 256, 4, 32, 0.01, 16, w_init="zeros", n_samples=2048),
    "mlr_mid": Workload("mlr_mid", MLR, 10_000, 20_000, 16, 64, 0.05, 50, zipf_s=1.1, x_scale="inv_sqrt_d"),
    "mlr_large": Workload("mlr_large", MLR, 325_000, 10_000, 16, 64, 0.05, 20, zipf_s=1.0,
                          x_scale="inv_sqrt_d"),
    "dml": Workload("dml", DML, 1_000, 20_000, 16, 64, 1e-3, 30, w_init="dml"),
    "sc": Workload("sc", SC, 10_000, 5_000, 16, 32, 1e-3, 20, w_init="unit_columns"),
}


def scaled(wl: Workload, name: str, **kw) -> Workload:
    """A reshaped copy of a workload (tests use small, ragged shapes with the same recipe)."""
    d = dict(wl.__dict__)
    d.update(kw)
    d["name"] = name
    return Workload(**d)


# ----------------------------------------------------------------------------------------------------------
# raw draws
# ----------------------------------------------------------------------------------------------------------
def _gen(seed: int, stream: int, block: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[np.uint64(seed), np.uint64((stream << 40) | block)]))


def _nblocks(rows: int) -> int:
    return (rows + _BLOCK_ROWS - 1) // _BLOCK_ROWS


def normal_rows(seed: int, stream: int, row0: int, row1: int, cols: int, scale: float = 1.0,
                out: np.ndarray | None = None) -> np.ndarray:
    """Rows ``[row0, row1)`` of the fp32 standard-normal matrix of stream ``stream`` (times ``scale``).

    ``row0`` must be a multiple of the block height; values are independent of how callers split the rows.
    """
    assert row0 % _BLOCK_ROWS == 0
    if out is None:
        out = np.empty((row1 - row0, cols), dtype=np.float32)
    sc = np.float32(scale)
    for b in range(row0 // _BLOCK_ROWS, _nblocks(row1)):
        r0 = b * _BLOCK_ROWS
        r1 = min(r0 + _BLOCK_ROWS, row1)
        blk = out[r0 - row0:r1 - row0]
        assert blk.flags.c_contiguous
        _gen(seed, stream, b).standard_normal(out=blk, dtype=np.float32)
        if sc != np.float32(1.0):
            np.multiply(blk, sc, out=blk)
    return out


def normal_matrix(seed: int, stream: int, rows: int, cols: int, scale: float = 1.0, threads: int = 8,
                  out: np.ndarray | None = None) -> np.ndarray:
    """The whole fp32 matrix of a stream, drawn block-parallel in ``threads`` threads."""
    if out is None:
        out = np.empty((rows, cols), dtype=np.float32)
    nb = _nblocks(rows)

    def work(b):
        r0 = b * _BLOCK_ROWS
        r1 = min(r0 + _BLOCK_ROWS, rows)
        normal_rows(seed, stream, r0, r1, cols, scale, out=out[r0:r1])

    if nb <= 1 or threads <= 1:
        for b in range(nb):
            work(b)
    else:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(work, range(nb)))
    return out


def zipf_labels(seed: int, stream: int, block: int, n: int, classes: int, s: float) -> np.ndarray:
    """``n`` int32 class ids with Pr(j) proportional to (j+1)^-s (s = 0: uniform), by inverse CDF in fp64."""
    u = _gen(seed, stream, block).random(n)
    if s == 0.0:
        return np.minimum((u * classes).astype(np.int64), classes - 1).astype(np.int32)
    w = np.arange(1, classes + 1, dtype=np.float64) ** (-s)
    cdf = np.cumsum(w)
    cdf /= cdf[-1]
    return np.minimum(np.searchsorted(cdf, u, side="right"), classes - 1).astype(np.int32)


# ----------------------------------------------------------------------------------------------------------
# per-workload inputs
# ----------------------------------------------------------------------------------------------------------
def initial_W(wl: Workload, threads: int = 8) -> np.ndarray:
    """W_0 as an fp32 row-major [rows x cols] array."""
    if wl.w_init == "zeros":
        return np.zeros((wl.rows, wl.cols), dtype=np.float32)
    if wl.w_init == "normal":
        return normal_matrix(wl.seed, _S_W0, wl.rows, wl.cols, wl.w_std, threads)
    if wl.w_init == "dml":
        return normal_matrix(wl.seed, _S_W0, wl.rows, wl.cols, 1.0 / math.sqrt(wl.cols), threads)
    if wl.w_init == "unit_columns":
        return _unit_columns(wl.seed, _S_W0, wl.rows, wl.cols, threads)
    raise ValueError(wl.w_init)


def _unit_columns(seed, stream, rows, cols, threads):
    g = normal_matrix(seed, stream, rows, cols, 1.0, threads).astype(np.float64)
    g /= np.sqrt((g * g).sum(axis=0, keepdims=True))
    return g.astype(np.float32)


@dataclass
class StepInputs:
    """Inputs of one minibatch step: K samples laid out worker-major (sample i = p*B + b)."""
    X: np.ndarray                      # fp32 [K x in_dim]
    Y: np.ndarray | None = None        # DML partner fp32 [K x cols]
    labels: np.ndarray | None = None   # int32 [K]: MLR class id | DML 1 = similar, 0 = dissimilar


def step_inputs(wl: Workload, step: int, true_dictionary: np.ndarray | None = None) -> StepInputs:
    """The K samples of minibatch ``step`` (deterministic sweep; worker p owns rows [p*B, (p+1)*B))."""
    K, dim = wl.K, wl.in_dim
    if wl.model == MLR:
        if wl.n_samples:
            Xall, yall = _mlr_pool(wl)
            lo = (step * K) % wl.n_samples
            return StepInputs(X=Xall[lo:lo + K].copy(), labels=yall[lo:lo + K].copy())
        scale = 1.0 / math.sqrt(dim) if wl.x_scale == "inv_sqrt_d" else 1.0
        X = _step_normal(wl.seed, _S_X, step, K, dim, scale)
        y = zipf_labels(wl.seed, _S_LABEL, step, K, wl.rows, wl.zipf_s)
        return StepInputs(X=X, labels=y)
    if wl.model == DML:
        X = _step_normal(wl.seed, _S_X, step, K, dim, 1.0)
        Z = _step_normal(wl.seed, _S_Y, step, K, dim, 1.0)
        sim = (_gen(wl.seed, _S_LABEL, step).random(K) < 0.5).astype(np.int32)
        Y = np.where(sim[:, None] == 1, X + np.float32(wl.dml_pair_noise) * Z, Z).astype(np.float32)
        return StepInputs(X=X, Y=Y, labels=sim)
    if wl.model == SC:
        Wt = true_dictionary if true_dictionary is not None else sc_true_dictionary(wl)
        A = wl.cols
        codes = np.zeros((K, A), dtype=np.float64)
        g = _gen(wl.seed, _S_SUPPORT, step)
        vals = _gen(wl.seed, _S_CODEVAL, step).standard_normal((K, wl.sc_nnz))
        for i in range(K):
            codes[i, g.choice(A, size=min(wl.sc_nnz, A), replace=False)] = vals[i, :min(wl.sc_nnz, A)]
        noise = _step_normal(wl.seed, _S_NOISE, step, K, dim, wl.sc_noise)
        X = (codes @ Wt.astype(np.float64).T + noise).astype(np.float32)
        return StepInputs(X=X)
    raise ValueError(wl.model)


def sc_true_dictionary(wl: Workload, threads: int = 8) -> np.ndarray:
    """The dictionary the SC samples are synthesised from (an independent draw, not W_0)."""
    return _unit_columns(wl.seed, _S_WTRUE, wl.rows, wl.cols, threads)


def _step_normal(seed, stream, step, K, dim, scale):
    out = np.empty((K, dim), dtype=np.float32)
    _gen(seed, stream, step).standard_normal(out=out, dtype=np.float32)
    if scale != 1.0:
        np.multiply(out, np.float32(scale), out=out)
    return out


_POOLS: dict = {}


def _mlr_pool(wl: Workload):
    key = (wl.seed, wl.n_samples, wl.cols, wl.rows, wl.zipf_s)
    if key not in _POOLS:
        X = normal_matrix(wl.seed, _S_X, wl.n_samples, wl.cols, 1.0, 1)
        y = zipf_labels(wl.seed, _S_LABEL, 0, wl.n_samples, wl.rows, wl.zipf_s)
        _POOLS[key] = (X, y)
    return _POOLS[key]


# ----------------------------------------------------------------------------------------------------------
# Delivery delays for the stale-synchronous emulation (Section 4.1): delay[c][p][q] in [0, staleness] is how many clocks
# beyond the next one the factors worker p produced at clock c take to reach worker q (0 on the diagonal).
# ----------------------------------------------------------------------------------------------------------
_S_DELAY = 9


def ssp_delays(seed: int, clocks: int, workers: int, staleness: int) -> np.ndarray:
    g = _gen(seed, _S_DELAY, 0)
    d = g.integers(0, staleness + 1, size=(clocks, workers, workers), dtype=np.int64)
    for p in range(workers):
        d[:, p, p] = 0
    return d


def asp_delays(seed: int, clocks: int, workers: int, mean: float) -> np.ndarray:
    """Delays without a bound (asynchronous parallel execution): geometric with the given mean, 0 on the diagonal."""
    g = _gen(seed, _S_DELAY, 1)
    d = g.geometric(1.0 / (1.0 + mean), size=(clocks, workers, workers)).astype(np.int64) - 1
    for p in range(workers):
        d[:, p, p] = 0
    return d


# ----------------------------------------------------------------------------------------------------------
# Sparse features (Section "Experiments": the paper's data sets have sparse features).  tf-idf-like samples in
# compressed-sparse-row form: the number of non-zeros of a sample is Poisson around nnz_mean (at least 1), its columns
# are drawn without replacement with Pr(column of popularity rank r) proportional to (r+1)^-zipf_s (the popularity
# order is a seeded permutation of the columns), its values are log-normal and the sample is scaled to unit length.
# ----------------------------------------------------------------------------------------------------------
_S_SPARSE = 10


@dataclass
class SparseSamples:
    indptr: np.ndarray     # int64 [n + 1]
    indices: np.ndarray    # int32 [nnz], ascending within a sample
    values: np.ndarray     # fp32 [nnz]

    @property
    def nnz(self) -> int:
        return int(self.indptr[-1] - self.indptr[0])


def sparse_samples(seed: int, step: int, n: int, cols: int, nnz_mean: float, zipf_s: float = 1.0) -> SparseSamples:
    g = _gen(seed, _S_SPARSE, step)
    order = _gen(seed, _S_SPARSE, 1 << 30).permutation(cols)
    w = np.arange(1, cols + 1, dtype=np.float64) ** (-zipf_s)
    prob = np.empty(cols, dtype=np.float64)
    prob[order] = w / w.sum()
    counts = np.clip(g.poisson(nnz_mean, size=n), 1, cols).astype(np.int64)
    indptr = np.zeros(n + 1, dtype=np.int64)
    np.cumsum(counts, out=indptr[1:])
    indices = np.empty(int(indptr[-1]), dtype=np.int32)
    values = np.empty(int(indptr[-1]), dtype=np.float32)
    for i in range(n):
        c = np.sort(g.choice(cols, size=int(counts[i]), replace=False, p=prob))
        v = np.exp(0.5 * g.standard_normal(int(counts[i])))
        v /= math.sqrt(float(np.dot(v, v)))
        indices[indptr[i]:indptr[i + 1]] = c
        values[indptr[i]:indptr[i + 1]] = v
    return SparseSamples(indptr=indptr, indices=indices, values=values)


def densify(sp: SparseSamples, cols: int) -> np.ndarray:
    """The same samples as a dense fp32 [n x cols] array (zeros elsewhere)."""
    n = len(sp.indptr) - 1
    X = np.zeros((n, cols), dtype=np.float32)
    rows = np.repeat(np.arange(n), np.diff(sp.indptr))
    X[rows, sp.indices] = sp.values
    return X
