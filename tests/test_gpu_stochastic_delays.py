"""GPU parity of the stage-wise stochastic delay model (Appendix E) against the oracle: every microbatch differentiated on
the current weights, each stage applying its slice of the gradient of a microbatch a drawn number of steps back."""
import numpy as np
import pytest

import pm_inputs as I
from parity_util import run_gpu_pipeline, compare_params, is_encdec

pytestmark = pytest.mark.gpu


def oracle_stochastic(wl, params0, delays, n_steps):
    from oracle import recurrence
    hp = dict(optimizer=wl.optimizer, alpha=wl.alpha, beta1=wl.beta1, beta2=wl.beta2, eps=wl.eps, t1=wl.t1, K=wl.K, t2=wl.t2, D=wl.D)
    if wl.kind == "encoder":
        from oracle import transformer
        data = (lambda t: I.seq2seq_batch(wl, t)) if is_encdec(wl) else (lambda t: I.token_batch(wl, t))
        grad_fn = transformer.make_grad_fn(wl.stage_specs, data, wl.n_heads, wl.seq_len, wl.vocab, wl.compute)
        flat0 = params0
    else:
        from oracle.mlp import make_grad_fn
        teacher = I.teacher_params(wl)
        grad_fn = make_grad_fn([[spec.act for spec in stage] for stage in wl.stages], lambda t: I.batch(wl, t, teacher), wl.compute)
        flat0 = [[t for pair in stage for t in pair] for stage in params0]
    return recurrence.run_stochastic(flat0, delays, wl.tau_fwd, grad_fn, n_steps, hp)


def check_applied(book_applied, res):
    ref = {(t, i): (s, n) for (t, i, s, n) in res.book}
    assert book_applied == ref


@pytest.mark.parametrize("compute,opt,per_stage", [("f32", "sgdm", 2), ("f32", "adam", 1), ("bf16", "sgdm", 2), ("bf16", "adam", 1)])
def test_stochastic_delays_mlp(cuda_device, compute, opt, per_stage):
    f32 = compute == "f32"
    P, tau_max = 5, 6
    wl = I.mlp_workload("hog", P, 72 if f32 else 192, per_stage, "gelu", 33 if f32 else 40, compute=compute, optimizer=opt,
                        alpha=0.02 if opt == "sgdm" else 1e-3, K=5, D=0.5, steps=14 if (f32 and opt == "adam") else 24, seed=191005124 + 90)
    means = [4, 3, 2, 1, 1]
    wl.tau_fwd = means                                         # the delay T1 divides by: the mean of the stage's distribution
    delays = I.stochastic_delays(wl.seed, wl.steps, means, tau_max)
    assert max(max(d) for d in delays) == tau_max and min(min(d) for d in delays) == 0     # the whole ring is used
    params0 = I.init_stage_params(wl)
    res = oracle_stochastic(wl, params0, delays, wl.steps)
    applied = {}
    pipe, losses, _ = run_gpu_pipeline(wl, params0, wl.steps, loop_order="mb_major", delays=delays, tau_max=tau_max, book_applied=applied)
    check_applied(applied, res)
    np.testing.assert_allclose(losses, np.array(res.losses), rtol=2e-5 if f32 else 1e-3)
    compare_params(pipe, res, (2e-5 if opt == "adam" else 1e-5) if f32 else 2e-2)
    assert float(pipe.delta.abs().max()) == 0.0                # T2 has nothing to correct in this model


@pytest.mark.parametrize("compute", ["f32", "bf16"])
def test_stochastic_delays_encoder_decoder(cuda_device, compute):
    f32 = compute == "f32"
    wl = I.cfg5_small(compute=compute, n_enc=1, n_dec=1, d_model=32 if f32 else 64, d_ff=64 if f32 else 128, seq_len=8 if f32 else 16,
                      batch=2, vocab=40 if f32 else 96, steps=14)
    P, tau_max = wl.n_stages, 5
    means = [max(1, (P - i) // 3) for i in range(P)]
    wl.tau_fwd = means
    delays = I.stochastic_delays(wl.seed, wl.steps, means, tau_max)
    params0 = I.init_encoder_params(wl)
    res = oracle_stochastic(wl, params0, delays, wl.steps)
    applied = {}
    pipe, losses, _ = run_gpu_pipeline(wl, params0, wl.steps, loop_order="mb_major", delays=delays, tau_max=tau_max, book_applied=applied)
    check_applied(applied, res)
    np.testing.assert_allclose(losses, np.array(res.losses), rtol=2e-5 if f32 else 1e-3)
    compare_params(pipe, res, 2e-5 if f32 else 2e-2, per_stage=not f32)


def test_zero_delays_equal_the_synchronous_mode(cuda_device):
    """All delays zero: the same bits as microbatch-major order with tau = 0 (synchronous training)."""
    import torch
    wl = I.mlp_workload("hog0", 4, 192, 1, "relu", 40, compute="bf16", optimizer="adam", alpha=1e-3, K=5, D=0.5, steps=10,
                        seed=191005124 + 91)
    wl.tau_fwd = [0] * 4
    params0 = I.init_stage_params(wl)
    sync, l0, _ = run_gpu_pipeline(wl, params0, wl.steps, loop_order="mb_major", collect_book=False)
    stoch, l1, _ = run_gpu_pipeline(wl, params0, wl.steps, loop_order="mb_major", collect_book=False,
                                    delays=[[0] * 4] * wl.steps, tau_max=3)
    np.testing.assert_array_equal(l0, l1)
    assert torch.equal(sync.w, stoch.w) and torch.equal(sync.m, stoch.m) and torch.equal(sync.s, stoch.s)


def test_stochastic_delay_rules(cuda_device):
    import paper_1910_05124_b200 as pm
    wl = I.mlp_workload("t", 3, 64, 1, "relu", 8, compute="f32", steps=4, seed=9)
    params0 = I.init_stage_params(wl)
    with pytest.raises(pm.PipeMareError, match="PM_ERR_UNSUPPORTED"):
        pm.Pipeline(wl, params0, stochastic_tau_max=4)                               # tick-major order
    plain = pm.Pipeline(wl, params0, loop_order="mb_major")
    with pytest.raises(pm.PipeMareError, match="PM_ERR_STATE"):
        plain.pm_set_delays([0, 0, 0])
    pipe = pm.Pipeline(wl, params0, loop_order="mb_major", stochastic_tau_max=4)
    with pytest.raises(pm.PipeMareError, match="PM_ERR_INVALID_ARG"):
        pipe.pm_set_delays([0, 5, 0])
    # the gradient ring: tau_max + 1 copies of the grad arena on top of a queue-less ring (one weight version per stage)
    total = 3 * (64 * 64 + 64)
    assert pipe.ring_bytes - pm.Pipeline(wl, params0, loop_order="mb_major", stochastic_tau_max=1).ring_bytes == 3 * total * 4
