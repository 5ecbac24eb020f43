"""pm_config.materialize_backward: the update writes the T2-corrected backward weights into a slot of the version queue and
dgrad reads them as a plain operand.  The correction is the same arithmetic at another moment, so every arena must end with
the SAME BITS as with the default path, which forms the corrected weights inside the dgrad kernel."""
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


@pytest.mark.parametrize("compute,opt,per_stage", [("f32", "sgdm", 2), ("bf16", "sgdm", 2), ("bf16", "adam", 1)])
def test_materialized_backward_mlp_bit_identical(cuda_device, compute, opt, per_stage):
    f32 = compute == "f32"
    wl = I.mlp_workload("mat", 5, 72 if f32 else 192, per_stage, "gelu", 33 if f32 else 40, compute=compute, optimizer=opt,
                        alpha=0.02 if opt == "sgdm" else 1e-3, K=5, D=0.5, steps=18, seed=191005124 + 97)
    params0 = I.init_stage_params(wl)
    plain, l0, _ = run_gpu_pipeline(wl, params0, wl.steps, loop_order="mb_major", collect_book=False)
    mat, l1, book = run_gpu_pipeline(wl, params0, wl.steps, loop_order="mb_major", materialize=1)
    np.testing.assert_array_equal(l0, l1)
    assert_same_state(plain, mat, opt == "adam")
    assert float(mat.delta.abs().max()) > 0.0                               # T2 is at work
    res = run_oracle(wl, params0, wl.steps)
    ref = {(t, i): (vf, vb) for (t, i, vf, vb) in res.book}
    for key, (vf, vb) in book.items():
        assert (vf, vb) == ref[key]
    np.testing.assert_allclose(l1, np.array(res.losses), rtol=2e-5 if f32 else 1e-3)
    compare_params(mat, res, 1e-5 if f32 else 2e-2)


@pytest.mark.parametrize("variant", ["plain", "warmup", "n_micro"])
def test_materialized_backward_encoder_decoder_bit_identical(cuda_device, variant):
    """Pair-tile GEMMs and LayerNorm gains (read corrected from the small-tensor ring); with synchronous warm-up steps and
    with two microbatches per update."""
    wl = I.cfg5_small(compute="bf16", n_enc=1, n_dec=1, d_model=256, n_heads=4, d_ff=512, seq_len=128, batch=2, vocab=264, steps=12)
    kw = {}
    if variant == "warmup":
        kw["warmup"] = 4
    if variant == "n_micro":
        kw["n_micro"] = 2
        wl.tau_fwd = I.pipemare_delays(wl.n_stages, 2)[0]
    params0 = I.init_encoder_params(wl)
    plain, l0, _ = run_gpu_pipeline(wl, params0, wl.steps, loop_order="mb_major", collect_book=False, **kw)
    mat, l1, _ = run_gpu_pipeline(wl, params0, wl.steps, loop_order="mb_major", collect_book=False, materialize=1, **kw)
    np.testing.assert_array_equal(l0, l1)
    assert_same_state(plain, mat, True)


def test_materialized_backward_rules(cuda_device):
    import paper_1910_05124_b200 as pm
    wl = I.mlp_workload("t", 3, 64, 1, "relu", 8, compute="bf16", steps=4, seed=9)
    params0 = I.init_stage_params(wl)
    with pytest.raises(pm.PipeMareError, match="PM_ERR_UNSUPPORTED"):
        pm.Pipeline(wl, params0, materialize_backward=1)                      # tick-major order keeps no version queue
    with pytest.raises(pm.PipeMareError, match="PM_ERR_UNSUPPORTED"):
        pm.Pipeline(wl, params0, loop_order="mb_major", materialize_backward=1, recompute_segment=2)
    a = pm.Pipeline(wl, params0, loop_order="mb_major")
    b = pm.Pipeline(wl, params0, loop_order="mb_major", materialize_backward=1)
    # per stage one more bf16 copy of its slice (4160 elements, the ring padded to 256 bytes) and an fp32 copy of its bias
    assert b.ring_bytes - a.ring_bytes == 3 * (8448 + 64 * 4)
