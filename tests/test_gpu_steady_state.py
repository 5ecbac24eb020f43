"""Parity in steady state at the configured widths: every stage past its pipeline fill, ring slots wrapping, every
forward reading a weight version that is tau_i updates old, and the grouped launch over all stages' tiles that the
benchmark times.  The microbatch is cut to fewer sequences (the GEMMs still have at least 256 rows, so the CTA-pair
kernels run) so that the oracle finishes 2P + 8 steps in a few minutes."""
import numpy as np
import pytest

import pm_inputs as I
from parity_util import run_gpu_pipeline, run_oracle, compare_params, compare_params_adam

pytestmark = pytest.mark.gpu


def check_book(book, res, n_steps, P):
    ref = {(t, i): (vf, vb) for (t, i, vf, vb) in res.book}
    assert len(book) == n_steps * P
    for key, (vf, vb) in book.items():
        assert (vf, vb) == ref[key], f"microbatch/stage {key}: device ({vf},{vb}) oracle {ref[key]}"


def test_cfg4_widths_all_stages_steady_state(cuda_device):
    """Config 4's 25 stages at its widths (d_model 512, 8 heads, FFN 2048, vocabulary 8192, sequences of 128 tokens),
    8 sequences per microbatch, 2P + 8 = 58 microbatches: stage 1 reads versions up to 8 through a 50-slot ring."""
    full = I.cfg4()
    wl = I.encoder_workload("cfg4_widths_8seq", 6, 512, 8, 2048, 128, 8, 8192, compute="bf16", optimizer="adam", alpha=full.alpha,
                            beta1=0.9, beta2=0.98, eps=1e-8, K=full.K, D=full.D, steps=2 * 25 + 8, seed=full.seed)
    assert wl.n_stages == 25
    params0 = I.init_encoder_params(wl)
    res = run_oracle(wl, params0, wl.steps)
    pipe, losses, book = run_gpu_pipeline(wl, params0, wl.steps)
    check_book(book, res, wl.steps, wl.n_stages)
    assert max(vf for (_, _, vf, _) in res.book) >= 8 and min(vf for (t, i, vf, _) in res.book if t == wl.steps - 1) >= 8
    print("cfg4 widths steady state: max loss relative error", np.abs(losses / np.array(res.losses) - 1).max())
    np.testing.assert_allclose(losses, np.array(res.losses), rtol=1e-3)
    rep = {}
    try:
        compare_params(pipe, res, 1e9, report=rep)              # report only: the max-norm measures, per tensor and per stage vector
    finally:
        print("cfg4 widths steady state max-norm weight errors", rep)
    print("cfg4 widths steady state weight errors", compare_params_adam(pipe, res, wl.steps))


def test_cfg5_widths_steady_state_both_orders(cuda_device):
    """Config 5's stage kinds at its widths (d_model 1024, 16 heads, FFN 4096, vocabulary 32000, sequences of 256
    tokens) on 2 + 2 layers (23 stages), 2 sequences per microbatch, 2P + 4 = 50 microbatches, in both loop orders."""
    wl = I.cfg5_cut(2, 2, batch=2)
    wl.steps = 2 * wl.n_stages + 4
    params0 = I.init_encoder_params(wl)
    res = run_oracle(wl, params0, wl.steps)
    for order in ("tick_major", "mb_major"):
        pipe, losses, book = run_gpu_pipeline(wl, params0, wl.steps, loop_order=order)
        check_book(book, res, wl.steps, wl.n_stages)
        print("cfg5 widths steady state", order, "max loss relative error", np.abs(losses / np.array(res.losses) - 1).max())
        np.testing.assert_allclose(losses, np.array(res.losses), rtol=1e-3)
        rep = {}
        try:
            compare_params(pipe, res, 1e9, report=rep)
        finally:
            print("cfg5 widths steady state", order, "max-norm weight errors", rep)
        print("cfg5 widths steady state", order, "weight errors", compare_params_adam(pipe, res, wl.steps))
        pipe.close()


def test_cfg5_widths_recompute_steady_state(cuda_device):
    """PipeMare Recompute at config 5's widths on 2 + 2 layers (23 stages), segments of 5 stages (boundaries inside
    layers: skip tensors, the memory and the main stream cross them), 2 sequences per microbatch, 32 microbatches (every
    recompute delay, at most 9 here, is past its clamp after ten; the forward delays' steady state is the test above):
    the pair-tile kernels, the 256-token attention, one weight-gradient launch per segment, T2-corrected recompute
    weights read from the queue."""
    wl = I.cfg5_cut(2, 2, batch=2)
    wl.steps = 32
    params0 = I.init_encoder_params(wl)
    res = run_oracle(wl, params0, wl.steps, segment=5)
    book_r = {}
    pipe, losses, book = run_gpu_pipeline(wl, params0, wl.steps, loop_order="mb_major", segment=5, book_recomp=book_r)
    check_book(book, res, wl.steps, wl.n_stages)
    ref_r = {(t, i): vr for (t, i, vr) in res.book_recomp}
    assert book_r == ref_r
    assert max(vr for vr in ref_r.values()) > 0 and any(ref_r[k] != res_v for k, res_v in ((k, v[0]) for k, v in book.items()))
    print("cfg5 widths recompute: max loss relative error", np.abs(losses / np.array(res.losses) - 1).max())
    np.testing.assert_allclose(losses, np.array(res.losses), rtol=1e-3)
    print("cfg5 widths recompute weight errors", compare_params_adam(pipe, res, wl.steps))
    pipe.close()


def test_adam_noise_evidence_at_config4_widths(cuda_device):
    """Oracle arithmetic only (it sits here because it needs the GPU machine's host cores for a minute): the oracle
    against a copy of itself whose gradients carry a relative perturbation of 2^-20, config 4's 25 stages at its
    widths, 58 updates.  Some entry of a weight matrix ends more than 2e-2 of the matrix's largest entry away, so a
    per-tensor max-norm of 2e-2 cannot be asked of any second implementation; the relative L2 difference and the
    fraction of entries beyond 2e-2 stay small, which is what compare_params_adam holds the GPU to."""
    from test_tolerance_evidence import adam_noise_experiment
    worst, (l2, frac, walk), loss_diff = adam_noise_experiment(6, 58)
    print("oracle vs perturbed oracle: worst per-tensor max-norm", worst, "L2", l2, "fraction beyond 2e-2", frac,
          "of the Adam walk", walk, "loss", loss_diff)
    assert worst > 2e-2 and l2 < 2e-2 and frac < 0.01 and loss_diff < 1e-3
