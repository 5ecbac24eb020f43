"""GPU parity of PipeMare Recompute (Appendix A.2, Appendix D) against the oracle: segment-wise recomputation with the
weights of its own delay, T2-corrected, in microbatch-major order."""
import numpy as np
import pytest

import pm_inputs as I
from parity_util import run_gpu_pipeline, run_oracle, compare_params, compare_params_adam, max_rel_err

pytestmark = pytest.mark.gpu


def check_books(book, book_r, res, n_steps, P):
    ref = {(t, i): (vf, vb) for (t, i, vf, vb) in res.book}
    assert len(book) == n_steps * P
    for key, (vf, vb) in book.items():
        assert (vf, vb) == ref[key], f"microbatch/stage {key}: device ({vf},{vb}) oracle {ref[key]}"
    ref_r = {(t, i): vr for (t, i, vr) in res.book_recomp}
    assert len(book_r) == n_steps * P
    for key, vr in book_r.items():
        assert vr == ref_r[key], f"microbatch/stage {key}: recompute version {vr}, oracle {ref_r[key]}"


@pytest.mark.parametrize("P,S,width,T,act,opt,t2", [
    (6, 2, 40, 7, "gelu", "sgdm", True),
    (7, 3, 72, 33, "relu", "sgdm", True),
    (5, 2, 64, 16, "relu", "adam", True),
    (6, 3, 48, 9, "gelu", "sgdm", False),
    (4, 1, 40, 8, "relu", "sgdm", True),
])
def test_recompute_fp32_mlp(cuda_device, P, S, width, T, act, opt, t2):
    wl = I.mlp_workload("rc", P, width, 1, act, T, compute="f32", optimizer=opt, alpha=0.05 if opt == "sgdm" else 1e-3,
                        K=6, D=0.5, steps=2 * P + 6, seed=191005124 + 70 + P)
    wl.t2 = t2
    params0 = I.init_stage_params(wl)
    res = run_oracle(wl, params0, wl.steps, segment=S)
    plain = run_oracle(wl, params0, wl.steps)
    book_r = {}
    pipe, losses, book = run_gpu_pipeline(wl, params0, wl.steps, loop_order="mb_major", segment=S, book_recomp=book_r)
    check_books(book, book_r, res, wl.steps, P)
    np.testing.assert_allclose(losses, np.array(res.losses), rtol=2e-5)
    tol = 2e-5 if opt == "adam" else 1e-5
    compare_params(pipe, res, tol)
    if S > 1:
        # the recomputation matters: without it the weights end far outside the tolerance of the comparison above
        moved = max(max_rel_err(a, b) for sa, sb in zip(res.params, plain.params) for a, b in zip(sa, sb))
        print("recompute vs none: largest relative weight difference", moved)
        assert moved > 50 * tol


@pytest.mark.parametrize("opt", ["sgdm", "adam"])
def test_recompute_bf16_mlp_with_several_linears_per_stage(cuda_device, opt):
    wl = I.mlp_workload("rc16", 6, 192, 2, "gelu", 40, compute="bf16", optimizer=opt, alpha=0.02 if opt == "sgdm" else 1e-3,
                        K=5, D=0.5, steps=20, seed=191005124 + 77)
    params0 = I.init_stage_params(wl)
    res = run_oracle(wl, params0, wl.steps, segment=2)
    book_r = {}
    pipe, losses, book = run_gpu_pipeline(wl, params0, wl.steps, loop_order="mb_major", segment=2, book_recomp=book_r)
    check_books(book, book_r, res, wl.steps, 6)
    np.testing.assert_allclose(losses, np.array(res.losses), rtol=1e-3)
    compare_params(pipe, res, 2e-2)


@pytest.mark.parametrize("compute,S", [("f32", 4), ("f32", 7), ("bf16", 4), ("bf16", 5)])
def test_recompute_encoder_decoder(cuda_device, compute, S):
    """Segments that cut through layers: skip tensors, the memory and the main stream cross segment boundaries as the
    forward pass left them; inside a segment they are recomputed."""
    f32 = compute == "f32"
    wl = I.cfg5_small(compute=compute, n_enc=2, n_dec=2, d_model=32 if f32 else 64, d_ff=64 if f32 else 128, seq_len=8 if f32 else 16,
                      batch=2, vocab=40 if f32 else 96, steps=14)
    params0 = I.init_encoder_params(wl)
    res = run_oracle(wl, params0, wl.steps, segment=S)
    book_r = {}
    pipe, losses, book = run_gpu_pipeline(wl, params0, wl.steps, loop_order="mb_major", segment=S, book_recomp=book_r)
    check_books(book, book_r, res, wl.steps, wl.n_stages)
    np.testing.assert_allclose(losses, np.array(res.losses), rtol=2e-5 if f32 else 1e-3)
    worst = compare_params(pipe, res, 2e-5 if f32 else 2e-2, per_stage=not f32)
    print("recompute encoder-decoder", compute, "S", S, "worst relative weight error", worst)


def test_recompute_tensor_core_path(cuda_device):
    """Pair-tile GEMMs and tensor-core attention, one weight-gradient launch per segment."""
    wl = I.cfg5_small(compute="bf16", n_enc=1, n_dec=1, d_model=256, n_heads=4, d_ff=512, seq_len=128, batch=2, vocab=264, steps=14)
    params0 = I.init_encoder_params(wl)
    res = run_oracle(wl, params0, wl.steps, segment=4)
    book_r = {}
    pipe, losses, book = run_gpu_pipeline(wl, params0, wl.steps, loop_order="mb_major", segment=4, book_recomp=book_r)
    check_books(book, book_r, res, wl.steps, wl.n_stages)
    np.testing.assert_allclose(losses, np.array(res.losses), rtol=1e-3)
    # bf16 operands and Adam: the criterion that knows Adam's +-alpha walk of elements whose gradient is rounding noise
    worst = compare_params_adam(pipe, res, wl.steps)
    print("recompute tc weight errors", worst)


@pytest.mark.parametrize("compute", ["f32", "bf16"])
def test_recompute_with_warmup_and_n_microbatches(cuda_device, compute):
    f32 = compute == "f32"
    P, N = 6, 2
    wl = I.mlp_workload("rcw", P, 64 if f32 else 192, 1, "gelu", 16 if f32 else 40, compute=compute, optimizer="sgdm",
                        alpha=0.01, K=5, D=0.5, steps=18, seed=191005124 + 78)
    params0 = I.init_stage_params(wl)
    res = run_oracle(wl, params0, wl.steps, warmup=4, segment=3)
    book_r = {}
    pipe, losses, book = run_gpu_pipeline(wl, params0, wl.steps, loop_order="mb_major", warmup=4, segment=3, book_recomp=book_r)
    check_books(book, book_r, res, wl.steps, P)
    np.testing.assert_allclose(losses, np.array(res.losses), rtol=2e-5 if f32 else 1e-3)
    compare_params(pipe, res, 1e-5 if f32 else 2e-2)
    # N microbatches per update: delays count updates (Table 1 with N; inside a segment likewise)
    wl.tau_fwd = I.pipemare_delays(P, N)[0]
    res = run_oracle(wl, params0, 6 * N + 1, n_micro=N, segment=3)
    book_r = {}
    pipe, losses, book = run_gpu_pipeline(wl, params0, 6 * N + 1, loop_order="mb_major", n_micro=N, segment=3, book_recomp=book_r)
    check_books(book, book_r, res, 6 * N + 1, P)
    np.testing.assert_allclose(losses, np.array(res.losses), rtol=2e-5 if f32 else 1e-3)
    compare_params(pipe, res, 1e-5 if f32 else 2e-2)


def test_recompute_rules(cuda_device):
    import paper_1910_05124_b200 as pm
    wl = I.mlp_workload("t", 4, 64, 1, "relu", 8, compute="f32", steps=4, seed=9)
    params0 = I.init_stage_params(wl)
    with pytest.raises(pm.PipeMareError, match="PM_ERR_UNSUPPORTED"):
        pm.Pipeline(wl, params0, recompute_segment=2)                         # tick-major order has one live version
    # one segment covering the pipeline is the plain method; the queue of corrected recompute weights costs ring bytes
    def q(S):
        pipe = pm.Pipeline(wl, params0, loop_order="mb_major", recompute_segment=S)
        sizes = (pipe.state_bytes, pipe.ring_bytes)
        pipe.close()
        return sizes
    assert q(4) == q(0) and q(9) == q(0)
    # stages 1, 2 keep tau_recomp + 1 = 4, 2 corrected versions of their 64 x 64 + 64 fp32 parameters (padded to 64)
    assert q(2)[1] - q(0)[1] == (4 + 2) * (64 * 64 + 64) * 4
