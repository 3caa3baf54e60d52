"""The prox entry point that allocates nothing, against the existing path.

Some callers of this library may not allocate device memory at all: code embedded in another program's fixed
memory budget, or a loop that cannot take the device-wide stall an allocation can cause.  They cannot create an
``sfb_ctx`` (it needs a workspace), so ``sfb_prox_columns_noalloc`` gives them the sparse-coding column prox
with its scratch in an array built into the library.  This file checks that entry point, through the C ABI,
against what the existing entry point (``sfb_step`` of a sparse-coding context, which ends with the same prox)
leaves in W -- twice in a row, with a different shape the second time, because every call shares the one built-in
array and must not depend on what the call before left there.

The file sorts last on purpose: a run that stops at the first failure has then already run every other test.
"""
import gc

import numpy as np
import pytest

import paper_1409_5705_b200 as S
import sfb_inputs as I
from oracle import sfb_oracle as O
from _parity import config_for, to_dev

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def _matrix(rows, cols, seed_stream):
    """Columns with norms on both sides of 1, so that some are rescaled and some must stay bit-identical."""
    W = I.normal_matrix(0, seed_stream, rows, cols, 1.0)
    norms = np.linalg.norm(W.astype(np.float64), axis=0)
    target = np.linspace(0.4, 1.9, cols)
    return (W * (target / norms)[None, :]).astype(np.float32)


def _existing_path(W0):
    """prox(W0) through the existing entry point: one sparse-coding step with eta = 0 adds exactly nothing to W
    and then applies the prox."""
    rows, cols = W0.shape
    wl = I.scaled(I.WORKLOADS["sc"], "sc_prox_only", rows=rows, cols=cols, workers=2, batch=4, eta=0.0, sc_nnz=3)
    inp = I.step_inputs(wl, 0, I.sc_true_dictionary(wl))
    W = to_dev(W0, torch)
    ctx = S.Context(config_for(wl, S.PREC_FP32, L=float(np.float32(O.lipschitz_power_iteration(W0)))), W)
    ctx.sfb_step(to_dev(inp.X, torch), None, None)
    assert ctx.sfb_get_status() == 0
    out = W.cpu().numpy()
    ctx.close()
    return out


def test_no_alloc_prox_matches_the_existing_entry_point_twice_in_a_row():
    for call, (rows, cols, stream) in enumerate([(300, 200, 21), (517, 1028, 22)]):
        W0 = _matrix(rows, cols, stream)
        expected = _existing_path(W0)
        W = to_dev(W0, torch)
        gc.collect()                                        # tensors of earlier tests are gone before we count
        if call == 0:
            # the very first call on a device may make the CUDA runtime load the library's device code (the built-in
            # array included): warm that up on a scratch copy so that the counters below see a steady state
            S.sfb_prox_columns_noalloc(W.clone())
            torch.cuda.synchronize()
        before = torch.cuda.memory_allocated()
        free_before = torch.cuda.mem_get_info()[0]          # the driver's own count: sees a cudaMalloc torch cannot
        S.sfb_prox_columns_noalloc(W)                       # the C-ABI call under test
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() <= before      # nothing was taken from torch's pool either
        assert torch.cuda.mem_get_info()[0] >= free_before  # and no device memory was taken behind torch's back
        got = W.cpu().numpy()
        # same kernels, same slab partition: the two paths agree to the last bit; 1e-5 is the suite's fp32 bound
        ref = O.prox_unit_columns(W0)
        den = np.linalg.norm(ref - W0.astype(np.float64))
        assert np.linalg.norm(got.astype(np.float64) - expected.astype(np.float64)) / den <= 1e-5, f"call {call}"
        np.testing.assert_array_equal(got, expected)
        # and both are the prox the oracle defines: norms <= 1, small columns untouched
        assert np.linalg.norm(got.astype(np.float64) - ref) / den <= 1e-5
        small = np.linalg.norm(W0.astype(np.float64), axis=0) <= 1.0
        np.testing.assert_array_equal(got[:, small], W0[:, small])


def test_no_alloc_prox_refuses_sizes_beyond_its_built_in_array():
    W = torch.zeros((4, S.NOALLOC_MAX_COLS + 4), dtype=torch.float32, device="cuda")
    with pytest.raises(S.SfbError) as e:
        S.sfb_prox_columns_noalloc(W)
    assert e.value.code == -11 and "built-in" in str(e.value)
    assert S.lib().sfb_prox_columns_noalloc(None, 4, 4, None) == -1
    assert (W == 0).all()
