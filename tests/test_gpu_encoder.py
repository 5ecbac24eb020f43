"""GPU parity of the Transformer-encoder pipeline (embedding, LayerNorm, attention, residuals, cross-entropy)."""
import numpy as np
import pytest

import pm_inputs as I
from parity_util import run_gpu_pipeline, run_oracle, compare_params

pytestmark = pytest.mark.gpu


def check_book(book, res, n_steps, P):
    ref = {(t, i): (vf, vb) for (t, i, vf, vb) in res.book}
    assert len(book) == n_steps * P
    for key, (vf, vb) in book.items():
        assert (vf, vb) == ref[key]


@pytest.mark.parametrize("kw", [
    dict(n_layers=1, d_model=32, n_heads=2, d_ff=64, seq_len=8, batch=2, vocab=40, steps=12),
    dict(n_layers=2, d_model=64, n_heads=4, d_ff=136, seq_len=16, batch=3, vocab=96, steps=24),
])
def test_encoder_fp32(cuda_device, kw):
    wl = I.cfg4_small(compute="f32", **kw)
    params0 = I.init_encoder_params(wl)
    res = run_oracle(wl, params0, wl.steps)
    pipe, losses, book = run_gpu_pipeline(wl, params0, wl.steps)
    check_book(book, res, wl.steps, wl.n_stages)
    np.testing.assert_allclose(losses, np.array(res.losses), rtol=2e-5)
    worst = compare_params(pipe, res, 2e-5)
    print("encoder fp32 worst relative weight error", worst)


@pytest.mark.parametrize("d_model", [328, 776])
def test_encoder_fp32_wide_rows(cuda_device, d_model):
    """LayerNorm rows of two 256-column groups with a ragged last group (328), and rows shared by two warps with a
    ragged second half (776).  SGD with momentum: with hundreds of thousands of weights some gradient sums cancel
    to rounding level, and Adam would turn the sign of such a sum into a step of alpha on either side."""
    wl = I.encoder_workload("wide_rows", 1, d_model, 2, 64, 8, 9, 60, compute="f32", optimizer="sgdm", alpha=0.02,
                            beta1=0.9, K=3, D=0.1, steps=10, seed=191005124 + 46)
    params0 = I.init_encoder_params(wl)
    res = run_oracle(wl, params0, wl.steps)
    pipe, losses, book = run_gpu_pipeline(wl, params0, wl.steps)
    check_book(book, res, wl.steps, wl.n_stages)
    np.testing.assert_allclose(losses, np.array(res.losses), rtol=2e-5)
    worst = compare_params(pipe, res, 2e-5)
    print("encoder fp32 wide rows worst relative weight error", worst)


@pytest.mark.parametrize("compute,vocab", [("f32", 8200), ("bf16", 8200), ("f32", 8198)])
def test_long_logit_rows(cuda_device, compute, vocab):
    """Vocabularies beyond 8192: the cross-entropy kernel that keeps the row of logits in shared memory (row lengths
    that are multiples of four) and the plain three-pass path (8198).  SGD with momentum, see the wide-row test."""
    wl = I.encoder_workload("long_rows", 1, 32, 2, 64, 8, 3, vocab, compute=compute, optimizer="sgdm", alpha=0.02,
                            beta1=0.9, K=3, D=0.1, steps=10, seed=191005124 + 47)
    params0 = I.init_encoder_params(wl)
    res = run_oracle(wl, params0, wl.steps)
    pipe, losses, book = run_gpu_pipeline(wl, params0, wl.steps)
    check_book(book, res, wl.steps, wl.n_stages)
    f32 = compute == "f32"
    np.testing.assert_allclose(losses, np.array(res.losses), rtol=2e-5 if f32 else 1e-3)
    worst = compare_params(pipe, res, 2e-5 if f32 else 2e-2, per_stage=not f32)
    print("long logit rows", compute, vocab, "worst relative weight error", worst)


def test_encoder_bf16_small(cuda_device):
    wl = I.cfg4_small(compute="bf16")
    params0 = I.init_encoder_params(wl)
    res = run_oracle(wl, params0, wl.steps)
    pipe, losses, book = run_gpu_pipeline(wl, params0, wl.steps)
    check_book(book, res, wl.steps, wl.n_stages)
    print("encoder bf16 loss errors", np.abs(losses / np.array(res.losses) - 1).max())
    np.testing.assert_allclose(losses, np.array(res.losses), rtol=1e-3)
    worst = compare_params(pipe, res, 2e-2, per_stage=True)
    print("encoder bf16 worst relative weight error (per stage vector)", worst)


def test_cfg4_full_size_first_microbatches(cuda_device):
    """Config 4 at its full size (6 layers, d_model 512, 8 heads, FFN 2048, 32 sequences of 128 tokens,
    vocabulary 8192, 25 stages): two microbatches fed and drained, so every stage has applied two updates."""
    wl = I.cfg4()
    n = 2
    params0 = I.init_encoder_params(wl)
    res = run_oracle(wl, params0, n)
    pipe, losses, book = run_gpu_pipeline(wl, params0, n)
    check_book(book, res, n, wl.n_stages)
    print("cfg4 loss relative errors", np.abs(losses / np.array(res.losses) - 1))
    np.testing.assert_allclose(losses, np.array(res.losses), rtol=1e-3)
    worst = compare_params(pipe, res, 2e-2, per_stage=True)
    print("cfg4 full size worst relative weight error (per stage vector)", worst)


def test_encoder_tensor_core_attention_shape(cuda_device):
    """Sequences of 128 tokens and heads of width 64 take the tensor-core attention kernels; everything else in
    this workload is small, so the oracle finishes quickly."""
    wl = I.cfg4_small(compute="bf16", n_layers=2, d_model=128, n_heads=2, d_ff=256, seq_len=128, batch=2, vocab=200, steps=12)
    params0 = I.init_encoder_params(wl)
    res = run_oracle(wl, params0, wl.steps)
    pipe, losses, book = run_gpu_pipeline(wl, params0, wl.steps)
    check_book(book, res, wl.steps, wl.n_stages)
    print("tc attention loss errors", np.abs(losses / np.array(res.losses) - 1).max())
    np.testing.assert_allclose(losses, np.array(res.losses), rtol=1e-3)
    worst = compare_params(pipe, res, 2e-2, per_stage=True)
    print("tc attention worst relative weight error (per stage vector)", worst)


# ---- encoder-decoder stages: causal self-attention, cross-attention over the encoder memory, two-stage skips ----------

@pytest.mark.parametrize("kw", [dict(n_enc=1, n_dec=1), dict(n_enc=2, n_dec=2, d_model=32, d_ff=64, seq_len=8, batch=2, vocab=40, steps=14)])
def test_encoder_decoder_fp32(cuda_device, kw):
    wl = I.cfg5_small(compute="f32", **kw)
    params0 = I.init_encoder_params(wl)
    res = run_oracle(wl, params0, wl.steps)
    pipe, losses, book = run_gpu_pipeline(wl, params0, wl.steps)
    check_book(book, res, wl.steps, wl.n_stages)
    np.testing.assert_allclose(losses, np.array(res.losses), rtol=2e-5)
    worst = compare_params(pipe, res, 2e-5)
    print("encoder-decoder fp32 worst relative weight error", worst)


def test_encoder_decoder_bf16_small(cuda_device):
    wl = I.cfg5_small(compute="bf16", n_enc=1, n_dec=2)
    params0 = I.init_encoder_params(wl)
    res = run_oracle(wl, params0, wl.steps)
    pipe, losses, book = run_gpu_pipeline(wl, params0, wl.steps)
    check_book(book, res, wl.steps, wl.n_stages)
    print("encoder-decoder bf16 loss errors", np.abs(losses / np.array(res.losses) - 1).max())
    np.testing.assert_allclose(losses, np.array(res.losses), rtol=1e-3)
    worst = compare_params(pipe, res, 2e-2, per_stage=True)
    print("encoder-decoder bf16 worst relative weight error (per stage vector)", worst)


def test_encoder_decoder_tensor_core_attention_shape(cuda_device):
    """Sequences of 128 tokens and heads of width 64: causal self-attention and cross-attention run on the
    tensor-core kernels."""
    wl = I.cfg5_small(compute="bf16", n_enc=1, n_dec=1, d_model=128, n_heads=2, d_ff=256, seq_len=128, batch=2, vocab=200, steps=10)
    params0 = I.init_encoder_params(wl)
    res = run_oracle(wl, params0, wl.steps)
    pipe, losses, book = run_gpu_pipeline(wl, params0, wl.steps)
    check_book(book, res, wl.steps, wl.n_stages)
    print("enc-dec tc attention loss errors", np.abs(losses / np.array(res.losses) - 1).max())
    np.testing.assert_allclose(losses, np.array(res.losses), rtol=1e-3)
    worst = compare_params(pipe, res, 2e-2, per_stage=True)
    print("enc-dec tc attention worst relative weight error (per stage vector)", worst)


def test_encoder_256_token_attention(cuda_device):
    """Sequences of 256 tokens (two blocks of 128 query rows per head) on the tensor-core attention kernels."""
    wl = I.cfg4_small(compute="bf16", n_layers=2, d_model=128, n_heads=2, d_ff=256, seq_len=256, batch=2, vocab=200, steps=10)
    params0 = I.init_encoder_params(wl)
    res = run_oracle(wl, params0, wl.steps)
    pipe, losses, book = run_gpu_pipeline(wl, params0, wl.steps)
    check_book(book, res, wl.steps, wl.n_stages)
    print("256-token attention loss errors", np.abs(losses / np.array(res.losses) - 1).max())
    np.testing.assert_allclose(losses, np.array(res.losses), rtol=1e-3)
    worst = compare_params(pipe, res, 2e-2, per_stage=True)
    print("256-token attention worst relative weight error (per stage vector)", worst)


def test_encoder_decoder_256_token_attention(cuda_device):
    """Config 5's own sequence length: causal self-attention and cross-attention over 256 tokens."""
    wl = I.cfg5_small(compute="bf16", n_enc=1, n_dec=1, d_model=128, n_heads=2, d_ff=256, seq_len=256, batch=2, vocab=200, steps=8)
    params0 = I.init_encoder_params(wl)
    res = run_oracle(wl, params0, wl.steps)
    pipe, losses, book = run_gpu_pipeline(wl, params0, wl.steps)
    check_book(book, res, wl.steps, wl.n_stages)
    print("enc-dec 256-token attention loss errors", np.abs(losses / np.array(res.losses) - 1).max())
    np.testing.assert_allclose(losses, np.array(res.losses), rtol=1e-3)
    worst = compare_params(pipe, res, 2e-2, per_stage=True)
    print("enc-dec 256-token attention worst relative weight error (per stage vector)", worst)


@pytest.mark.parametrize("shape", [dict(seq_len=256, batch=16), dict(seq_len=128, batch=32)])
def test_cfg5_widths_first_microbatches(cuda_device, shape):
    """Config 5's widths (d_model 1024, 16 heads, FFN 4096; 16 sequences of 256 tokens as the config has them, and
    32 of 128) on one encoder and one decoder layer with a vocabulary of 4096: two microbatches fed and drained.
    Every GEMM runs on the CTA-pair kernels, attention (self, causal, cross) on the tensor-core kernels."""
    wl = I.cfg5_cut(1, 1, vocab=4096, **shape)
    n = 2
    params0 = I.init_encoder_params(wl)
    res = run_oracle(wl, params0, n)
    pipe, losses, book = run_gpu_pipeline(wl, params0, n)
    check_book(book, res, n, wl.n_stages)
    print("cfg5 widths loss relative errors", np.abs(losses / np.array(res.losses) - 1))
    np.testing.assert_allclose(losses, np.array(res.losses), rtol=1e-3)
    worst = compare_params(pipe, res, 2e-2, per_stage=True)
    print("cfg5 widths worst relative weight error (per stage vector)", worst)


def _final_weights(wl, params0, n):
    pipe, losses, _ = run_gpu_pipeline(wl, params0, n, collect_book=False)
    import torch
    return pipe.w.clone(), torch.tensor(losses)


def test_runs_are_bit_reproducible_and_graph_replay_changes_nothing(cuda_device, monkeypatch):
    """Every reduction on the path has a fixed order (no floating-point atomics), so two runs of the same workload
    give the same bits; replaying the phases as CUDA graphs launches the same kernels and must give those bits too."""
    import torch
    wl = I.cfg5_small(compute="bf16", n_enc=1, n_dec=1, steps=12)
    params0 = I.init_encoder_params(wl)
    w_a, l_a = _final_weights(wl, params0, wl.steps)
    w_b, l_b = _final_weights(wl, params0, wl.steps)
    assert torch.equal(w_a, w_b) and torch.equal(l_a, l_b)
    monkeypatch.setenv("PM_CUDA_GRAPHS", "0")
    w_c, l_c = _final_weights(wl, params0, wl.steps)
    assert torch.equal(w_a, w_c) and torch.equal(l_a, l_c)
