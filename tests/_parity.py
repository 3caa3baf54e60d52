"""Helpers of the GPU parity tests: run one step through the C ABI, run the oracle on the same inputs,
and form the error ratio  ||W_gpu - W_ref||_F / ||W_ref - W_0||_F  (error of the stored W over the size of the update)."""
from __future__ import annotations

import numpy as np

import paper_1409_5705_b200 as S
import sfb_inputs as I
from oracle import sfb_oracle as O

TOL = {S.PREC_FP32: 1e-5, S.PREC_BF16: 2e-3, S.PREC_TF32X3: 1e-5, S.PREC_FP32_FFMA: 1e-5}


def config_for(wl: I.Workload, precision, L=0.0, prox=None):
    return S.make_config(wl.model, wl.rows, wl.cols, wl.workers, wl.batch, wl.eta, precision,
                         dml_margin=wl.dml_margin, sc_lambda=wl.sc_lambda, sc_ista_iters=wl.sc_iters,
                         sc_lipschitz=float(L), sc_prox=(1 if wl.model == I.SC else 0) if prox is None else prox)


def to_dev(a, torch):
    return None if a is None else torch.from_numpy(np.ascontiguousarray(a)).cuda()


def oracle_step(wl: I.Workload, W, inp: I.StepInputs, L=None, return_factors=False):
    return O.sfb_step(wl.model, W, inp.X, inp.Y, inp.labels, workers=wl.workers, eta=wl.eta,
                      margin=wl.dml_margin, lam=wl.sc_lambda, L=L, iters=wl.sc_iters, prox=(wl.model == I.SC),
                      return_factors=return_factors)


def rel_err(W_gpu, W_ref64, W0):
    """Error of the stored fp32 W against the oracle's W rounded once to fp32, over the size of the update."""
    ref32 = W_ref64.astype(np.float32).astype(np.float64)
    den = np.linalg.norm(W_ref64 - W0.astype(np.float64))
    return float(np.linalg.norm(W_gpu.astype(np.float64) - ref32) / den)


def entries_excess(W_gpu, W_ref64, W0, stores=1):
    """Largest entry-wise error beyond what storing W in fp32 `stores` times allows (half an fp32 spacing per store),
    in units of the rms entry of the update."""
    ref32 = np.abs(W_ref64).astype(np.float32)
    half_ulp = 0.5 * stores * np.spacing(ref32).astype(np.float64)
    upd = W_ref64 - W0.astype(np.float64)
    rms = float(np.sqrt((upd * upd).mean()))
    excess = np.abs(W_gpu.astype(np.float64) - W_ref64) - half_ulp
    return float(excess.max()) / rms


def entries_ok(W_gpu, W_ref64, W0, tol, stores=1):
    """Entry-wise check, for what a norm over the whole matrix can hide (rows whose update is only a few fp32 ulps
    of W, a ragged last tile): every stored entry must lie within half an fp32 spacing per store of the oracle's
    value, plus 8*tol times the rms entry of the update on those rows.  A missing or misplaced update (tens of
    ulps) fails it."""
    return entries_excess(W_gpu, W_ref64, W0, stores) <= 8 * tol


def storage_floor(W_ref64, W0):
    """||fl32(W_ref) - W_ref|| / ||W_ref - W_0||: the error any implementation that stores W in fp32 has
    against the unrounded oracle.  A step that stores W twice (update, then prox) pays it once more against
    the once-rounded reference, so sparse-coding steps are allowed 2*floor on top of the tolerance."""
    ref32 = W_ref64.astype(np.float32).astype(np.float64)
    return float(np.linalg.norm(ref32 - W_ref64) / np.linalg.norm(W_ref64 - W0.astype(np.float64)))


def step_tol(wl, prec, W_ref64, W0, prox=True):
    """Tolerance of one step: the stated bound, plus for sparse coding the storage floor once per extra store of W
    (with the prox the step stores W twice: twice the floor; without it once: one floor)."""
    extra = (2.0 if prox else 1.0) * storage_floor(W_ref64, W0) if wl.model == I.SC else 0.0
    return TOL[prec] + extra
