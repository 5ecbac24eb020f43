"""GPU parity of synchronous warm-up followed by PipeMare (PipeMareW, Section 4) against the oracle."""
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


@pytest.mark.parametrize("opt,warmup", [("sgdm", 5), ("adam", 5), ("sgdm", 14), ("adam", 1)])
def test_fp32_mlp_warmup_then_pipemare(cuda_device, opt, warmup):
    """Warm-up shorter than, equal to (14 = every step) and barely present (1) in a 14-step run; T1 with K = 6 is
    still annealing when PipeMare starts, T2 is on."""
    wl = I.mlp_workload("w", 4, 72, 2, "gelu", 24, compute="f32", optimizer=opt, alpha=0.01 if opt == "sgdm" else 1e-3,
                        K=6, D=0.5, steps=14, seed=191005124 + 81)
    params0 = I.init_stage_params(wl)
    res = run_oracle(wl, params0, wl.steps, warmup=warmup)
    pipe, losses, book = run_gpu_pipeline(wl, params0, wl.steps, warmup=warmup)
    check_book(book, res, wl.steps, wl.n_stages)
    np.testing.assert_allclose(losses, np.array(res.losses), rtol=2e-5)
    compare_params(pipe, res, 2e-5)
    # delta: zero while only warm-up steps have run, the oracle's values afterwards
    import torch
    got = pipe.unpack(pipe.delta)
    for p, stage in enumerate(got):
        for j, (W, b) in enumerate(stage):
            ref = res.delta[p][2 * j]
            if warmup >= wl.steps:
                assert not np.asarray(W).any() and not ref.any()
            else:
                # delta averages differences w' - w of nearly equal numbers: a few fp32 ulps of w show up at 1e-4 of delta's size
                np.testing.assert_allclose(W, ref, atol=3e-4 * max(np.abs(ref).max(), 1e-12))


def test_warmup_changes_the_trajectory(cuda_device):
    """The same run with and without warm-up ends at different weights (the test above would also pass if the flag
    did nothing on both sides)."""
    wl = I.mlp_workload("w", 3, 64, 1, "relu", 16, compute="f32", optimizer="sgdm", alpha=0.02, K=5, D=0.3, steps=10, seed=3)
    params0 = I.init_stage_params(wl)
    a, la, _ = run_gpu_pipeline(wl, params0, wl.steps, warmup=0, collect_book=False)
    b, lb, _ = run_gpu_pipeline(wl, params0, wl.steps, warmup=4, collect_book=False)
    assert la[0] == lb[0] and not np.array_equal(la, lb)
    import torch
    assert not torch.equal(a.w, b.w)


def test_bf16_encoder_decoder_warmup(cuda_device):
    wl = I.cfg5_small(compute="bf16", n_enc=1, n_dec=1, steps=12)
    params0 = I.init_encoder_params(wl)
    res = run_oracle(wl, params0, wl.steps, warmup=4)
    pipe, losses, book = run_gpu_pipeline(wl, params0, wl.steps, warmup=4)
    check_book(book, res, wl.steps, wl.n_stages)
    np.testing.assert_allclose(losses, np.array(res.losses), rtol=1e-3)
    worst = compare_params(pipe, res, 2e-2, per_stage=True)
    print("warm-up encoder-decoder bf16 worst relative weight error (per stage vector)", worst)


def test_warmup_feeding_rules(cuda_device):
    import torch
    import paper_1910_05124_b200 as pm
    wl = I.mlp_workload("t", 2, 64, 1, "relu", 8, compute="f32", steps=4, seed=9)
    pipe = pm.Pipeline(wl, I.init_stage_params(wl))
    x, y = I.batch(wl, 0)
    xd, yd = torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda()
    with pytest.raises(pm.PipeMareError, match="PM_ERR_INVALID_ARG"):
        pipe.pm_set_warmup(-1)
    pipe.pm_set_warmup(2)
    pipe.pm_step(xd, yd)                                       # tick 0: warm-up microbatch 0
    with pytest.raises(pm.PipeMareError, match="before the first tick"):
        pipe.pm_set_warmup(3)
    with pytest.raises(pm.PipeMareError, match="takes none"):
        pipe.pm_step(xd, yd)                                   # tick 1 lies between two warm-up microbatches
    for _ in range(3):
        pipe.pm_step(None, None)                               # ticks 1..3: not the end of the stream
    assert pipe.pm_get_losses(0, 1).shape == (1,)              # microbatch 0 finished after 2P - 1 = 3 more ticks
    pipe.pm_step(xd, yd)                                       # tick 4 = 2P: warm-up microbatch 1
    for _ in range(3):
        pipe.pm_step(None, None)
    pipe.pm_step(xd, yd)                                       # tick 8: first PipeMare microbatch
    pipe.pm_step(xd, yd)                                       # tick 9: one per tick from here on
    with pytest.raises(pm.PipeMareError, match="not finished"):
        pipe.pm_get_losses(0, 4)
    pipe.pm_step(None, None)
    with pytest.raises(pm.PipeMareError, match="draining"):
        pipe.pm_step(xd, yd)
    for _ in range(3):
        pipe.pm_step(None, None)
    assert pipe.pm_get_losses(0, 4).shape == (4,)
