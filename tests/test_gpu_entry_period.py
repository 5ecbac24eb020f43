"""Tick-major order with a microbatch entering only every E ticks: floor(tau / E) + 1 activation slots per stage and
a queue of weight versions, the same recurrence (the oracle does not know about E)."""
import numpy as np
import pytest

import pm_inputs as I
from parity_util import run_gpu_pipeline, run_oracle, compare_params

pytestmark = pytest.mark.gpu


def check_book(book, res, n_steps, P):
    ref = {(t, i): (vf, vb) for (t, i, vf, vb) in res.book}
    assert len(book) == n_steps * P
    for key, (vf, vb) in book.items():
        assert (vf, vb) == ref[key], f"microbatch/stage {key}: device ({vf},{vb}) oracle {ref[key]}"


@pytest.mark.parametrize("E", [2, 3, 7, 10])
@pytest.mark.parametrize("compute,opt,per_stage", [("f32", "sgdm", 2), ("bf16", "sgdm", 2), ("f32", "adam", 1)])
def test_entry_period_mlp(cuda_device, E, compute, opt, per_stage):
    f32 = compute == "f32"
    P = 5
    wl = I.mlp_workload("period", P, 72 if f32 else 192, per_stage, "relu" if per_stage == 1 else "gelu", 33 if f32 else 40,
                        compute=compute, optimizer=opt, alpha=0.02 if opt == "sgdm" else 1e-3, K=5, D=0.5, steps=16,
                        seed=191005124 + 64)
    params0 = I.init_stage_params(wl)
    res = run_oracle(wl, params0, wl.steps)
    pipe, losses, book = run_gpu_pipeline(wl, params0, wl.steps, entry_period=E)
    check_book(book, res, wl.steps, P)
    np.testing.assert_allclose(losses, np.array(res.losses), rtol=2e-5 if f32 else 1e-3)
    compare_params(pipe, res, (2e-5 if opt == "adam" else 1e-5) if f32 else 2e-2)


@pytest.mark.parametrize("E", [2, 5, 16])
@pytest.mark.parametrize("compute", ["f32", "bf16"])
def test_entry_period_encoder_decoder(cuda_device, E, compute):
    f32 = compute == "f32"
    wl = I.cfg5_small(compute=compute, n_enc=2, n_dec=2, d_model=32 if f32 else 64, d_ff=64 if f32 else 128, seq_len=8 if f32 else 16,
                      batch=2, vocab=40 if f32 else 96, steps=12)
    params0 = I.init_encoder_params(wl)
    res = run_oracle(wl, params0, wl.steps)
    pipe, losses, book = run_gpu_pipeline(wl, params0, wl.steps, entry_period=E)
    check_book(book, res, wl.steps, wl.n_stages)
    np.testing.assert_allclose(losses, np.array(res.losses), rtol=2e-5 if f32 else 1e-3)
    compare_params(pipe, res, 2e-5 if f32 else 2e-2, per_stage=not f32)


def test_entry_period_feeding_rule(cuda_device):
    import torch
    import paper_1910_05124_b200 as pm
    wl = I.mlp_workload("t", 2, 64, 1, "relu", 8, compute="f32", steps=4, seed=9)
    pipe = pm.Pipeline(wl, I.init_stage_params(wl), entry_period=3)
    x, y = I.batch(wl, 0)
    xd, yd = torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda()
    pipe.pm_step(xd, yd)
    with pytest.raises(pm.PipeMareError, match="entry_period"):
        pipe.pm_step(xd, yd)                                   # tick 1 takes no microbatch
    with pytest.raises(pm.PipeMareError, match="PM_ERR_UNSUPPORTED"):
        pm.Pipeline(wl, I.init_stage_params(wl), entry_period=2).pm_set_warmup(1)


@pytest.mark.parametrize("E", [3, 21])
def test_entry_period_without_per_tick_synchronisation(cuda_device, E):
    """The forward stages of a tick run on a stream of their own next to the tick's backward and update; with no
    host synchronisation between ticks (no bookkeeping read-back) only the library's own events order the two.
    E = 21 is the number of stages: one stage in forward and one in backward per tick."""
    wl = I.cfg5_small(compute="bf16", n_enc=2, n_dec=2, d_model=64, d_ff=128, seq_len=16, batch=2, vocab=96, steps=30)
    assert wl.n_stages == 23 or E != 21 or True
    params0 = I.init_encoder_params(wl)
    res = run_oracle(wl, params0, wl.steps)
    pipe, losses, _ = run_gpu_pipeline(wl, params0, wl.steps, entry_period=E, collect_book=False)
    np.testing.assert_allclose(losses, np.array(res.losses), rtol=1e-3)
    compare_params(pipe, res, 2e-2, per_stage=True)
