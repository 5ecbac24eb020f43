"""The update of the Linear matrices applied in the weight-gradient GEMM's epilogue (pm_config.fuse_update): the same
arithmetic per element as the stand-alone update kernel, so a fused run must end with the SAME BITS as an unfused one,
in every arena, and both match the oracle."""
import numpy as np
import pytest

import pm_inputs as I
from parity_util import run_gpu_pipeline, run_oracle, compare_params

pytestmark = pytest.mark.gpu


def assert_same_state(a, b, adam):
    import torch
    for name in ("w", "m", "delta") + (("s",) if adam else ()):
        x, y = getattr(a, name), getattr(b, name)
        assert torch.equal(x, y), f"arena {name}: {int((x != y).sum())} of {x.numel()} elements differ"
    if a.w_lp is not None and not a.mb_major:
        assert torch.equal(a.w_lp, b.w_lp)


@pytest.mark.parametrize("order", ["tick_major", "mb_major"])
@pytest.mark.parametrize("opt", ["sgdm", "adam"])
def test_fused_update_bf16_mlp_bit_identical(cuda_device, order, opt):
    # one Linear per stage, widths that are not multiples of the 256-wide tiles, a ragged last tile in both dimensions
    wl = I.mlp_workload("fu", 5, 328, 1, "gelu", 72, compute="bf16", optimizer=opt, alpha=0.02 if opt == "sgdm" else 1e-3,
                        K=5, D=0.5, steps=16, seed=191005124 + 81)
    params0 = I.init_stage_params(wl)
    res = run_oracle(wl, params0, wl.steps)
    plain, losses0, _ = run_gpu_pipeline(wl, params0, wl.steps, loop_order=order, collect_book=False)
    fused, losses1, book = run_gpu_pipeline(wl, params0, wl.steps, loop_order=order, fuse_update=1)
    np.testing.assert_array_equal(losses0, losses1)
    assert_same_state(plain, fused, opt == "adam")
    np.testing.assert_allclose(losses1, np.array(res.losses), rtol=1e-3)
    compare_params(fused, res, 2e-2)
    ref = {(t, i): (vf, vb) for (t, i, vf, vb) in res.book}
    for key, (vf, vb) in book.items():
        assert (vf, vb) == ref[key]                            # the update counters are still kept by the update kernel


@pytest.mark.parametrize("order", ["tick_major", "mb_major"])
def test_fused_update_encoder_decoder_bit_identical(cuda_device, order):
    """Pair-tile GEMMs (256-wide and wider Linears), LayerNorm parameters and embedding tables updated by the update kernel
    next to the matrices updated in the epilogue."""
    wl = I.cfg5_small(compute="bf16", n_enc=1, n_dec=1, d_model=256, n_heads=4, d_ff=512, seq_len=128, batch=2, vocab=264, steps=12)
    params0 = I.init_encoder_params(wl)
    plain, losses0, _ = run_gpu_pipeline(wl, params0, wl.steps, loop_order=order, collect_book=False)
    fused, losses1, _ = run_gpu_pipeline(wl, params0, wl.steps, loop_order=order, collect_book=False, fuse_update=1)
    np.testing.assert_array_equal(losses0, losses1)
    assert_same_state(plain, fused, True)
    res = run_oracle(wl, params0, wl.steps)
    np.testing.assert_allclose(losses1, np.array(res.losses), rtol=1e-3)
    compare_params(fused, res, 2e-2, per_stage=True)


def test_fused_update_with_warmup(cuda_device):
    wl = I.mlp_workload("fuw", 4, 256, 1, "relu", 64, compute="bf16", optimizer="adam", alpha=1e-3, K=5, D=0.5, steps=14,
                        seed=191005124 + 82)
    params0 = I.init_stage_params(wl)
    for order in ("tick_major", "mb_major"):
        plain, l0, _ = run_gpu_pipeline(wl, params0, wl.steps, loop_order=order, warmup=4, collect_book=False)
        fused, l1, _ = run_gpu_pipeline(wl, params0, wl.steps, loop_order=order, warmup=4, collect_book=False, fuse_update=1)
        np.testing.assert_array_equal(l0, l1)
        assert_same_state(plain, fused, True)


def test_fused_update_rules(cuda_device):
    import paper_1910_05124_b200 as pm
    wl = I.mlp_workload("t", 3, 64, 1, "relu", 8, compute="f32", steps=4, seed=9)
    with pytest.raises(pm.PipeMareError, match="PM_ERR_UNSUPPORTED"):
        pm.Pipeline(wl, I.init_stage_params(wl), fuse_update=1)                      # fp32 operands: no tensor-core epilogue
    wl2 = I.mlp_workload("t", 3, 64, 2, "relu", 8, compute="bf16", steps=4, seed=9)
    with pytest.raises(pm.PipeMareError, match="PM_ERR_UNSUPPORTED"):
        pm.Pipeline(wl2, I.init_stage_params(wl2), fuse_update=1)                    # several Linears per stage
    wl3 = I.mlp_workload("t", 3, 64, 1, "relu", 8, compute="bf16", steps=4, seed=9)
    with pytest.raises(pm.PipeMareError, match="PM_ERR_UNSUPPORTED"):
        pm.Pipeline(wl3, I.init_stage_params(wl3), loop_order="mb_major", n_micro=2, fuse_update=1)
