"""The operand copy of W that MLR keeps for its forward product must equal the rounding of the current W exactly,
step after step: the update rewrites only the row pieces whose bf16 rounding changed (the others already hold the
right bits), the label-row pass rewrites its rows, and the tensor-core fp32 mode rewrites its pair of tf32 words with
every entry.  Checked bit for bit after several steps, with steps so small that almost nothing changes in bf16 and
with steps large enough to change most of it."""
import numpy as np
import pytest

import paper_1409_5705_b200 as S
import sfb_inputs as I
from _parity import config_for, to_dev

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def _workload(eta):
    return I.scaled(I.WORKLOADS["mlr_mid"], "mlr_copy", rows=700, cols=516, workers=3, batch=50, eta=eta, w_std=0.05,
                    x_scale="unit")


@pytest.mark.parametrize("eta", [1e-6, 0.05, 20.0])
@pytest.mark.parametrize("prox", [0, 1])
def test_bf16_copy_equals_the_rounded_W_after_every_step(eta, prox):
    wl = _workload(eta)
    W = to_dev(I.initial_W(wl), torch)
    cfg = config_for(wl, S.PREC_BF16)
    cfg.prox_kind, cfg.prox_weight = prox, (0.01 / eta if prox else 0.0)
    ctx = S.Context(cfg, W)
    fractions = []
    for t in range(4):
        inp = I.step_inputs(wl, t)
        before = ctx.sfb_get_stats()
        ctx.sfb_step(to_dev(inp.X, torch), None, to_dev(inp.labels, torch))
        assert ctx.sfb_get_status() == 0
        copy = ctx.operand_copy_as_tensor()[:, :wl.cols]
        assert torch.equal(copy, W.to(torch.bfloat16)), f"step {t}"
        after = ctx.sfb_get_stats()
        fractions.append((after.copy_written - before.copy_written) / max(1, after.copy_pieces - before.copy_pieces))
    print(f"eta {eta} prox {prox}: fraction of row pieces rewritten per step", " ".join(f"{f:.3f}" for f in fractions))
    if eta <= 1e-6 and not prox:
        assert max(fractions) < 0.2                     # tiny steps: most pieces keep their bf16 bits
    if eta == 0.05:
        assert min(fractions) > 0.3                     # ordinary steps on this small, fast-moving case: many do change
    ctx.close()


def test_tf32_pair_copy_equals_the_split_of_W_after_every_step():
    wl = _workload(0.05)
    W = to_dev(I.initial_W(wl), torch)
    ctx = S.Context(config_for(wl, S.PREC_TF32X3), W)
    for t in range(3):
        inp = I.step_inputs(wl, t)
        ctx.sfb_step(to_dev(inp.X, torch), None, to_dev(inp.labels, torch))
        assert ctx.sfb_get_status() == 0
        copy = ctx.operand_copy_as_tensor()
        half = copy.shape[1] // 2
        big, small = copy[:, :wl.cols], copy[:, half:half + wl.cols]
        # big keeps the 10 explicit mantissa bits of tf32 (round to nearest, ties away); big + small restores W to 2^-22
        assert int((big.view(torch.int32) & 0x1FFF).abs().max()) == 0 and int((small.view(torch.int32) & 0x1FFF).abs().max()) == 0
        assert float((W - big).abs().max()) <= float(W.abs().max()) * 2.0 ** -11
        assert float(((W - big) - small).abs().max()) <= float(W.abs().max()) * 2.0 ** -21
    ctx.close()
