"""Pins for oracle/transformer.py: finite differences of the whole encoder (u_fwd = u_bkwd), two-argument semantics."""
import numpy as np
import pytest

import pm_inputs as I
from oracle import transformer as TR


def small(compute="f32"):
    wl = I.cfg4_small(compute=compute, n_layers=1, d_model=8, n_heads=2, d_ff=12, seq_len=4, batch=2, vocab=11)
    params = [[a.astype(np.float64) for a in st] for st in I.init_encoder_params(wl)]
    rng = np.random.default_rng(3)
    for st in params:                      # move biases and LayerNorm parameters off their special initial values
        for a in st:
            a += rng.normal(size=a.shape) * 0.1
    return wl, params


def test_stage_list_of_the_encoder():
    wl = I.cfg4()
    assert wl.n_stages == 25 and len(wl.stage_specs) == 25
    assert [s.post for s in wl.stage_specs[:4]] == ["attention", "residual", "skip_out", "residual"]
    assert wl.stage_specs[0].pre == "embed" and wl.stage_specs[4].pre == "ln" and wl.stage_specs[-1].n_out == 8192
    assert wl.tau_fwd[0] == 49 and wl.tau_fwd[-1] == 1
    ids, tg = I.token_batch(wl, 0)
    assert ids.shape == (4096,) and (ids.reshape(32, 128)[:, ::-1] == tg.reshape(32, 128)).all()


def test_encoder_gradients_match_central_differences():
    wl, params = small()
    data = I.token_batch(wl, 0)
    grad_fn = TR.make_grad_fn(wl.stage_specs, lambda t: data, wl.n_heads, wl.seq_len, wl.vocab, "f32")
    loss, g = grad_fn(0, params, params)
    h = 1e-6
    rng = np.random.default_rng(0)
    for i, st in enumerate(params):
        for j, a in enumerate(st):
            flat = a.reshape(-1)
            for idx in rng.choice(flat.size, size=min(6, flat.size), replace=False):
                old = flat[idx]
                flat[idx] = old + h
                lp, _ = grad_fn(0, params, params)
                flat[idx] = old - h
                lm, _ = grad_fn(0, params, params)
                flat[idx] = old
                fd = (lp - lm) / (2 * h)
                assert np.asarray(g[i][j]).reshape(-1)[idx] == pytest.approx(fd, rel=2e-5, abs=2e-9), (i, j, idx)


def test_backward_weights_enter_only_through_linear_dgrad_and_layernorm_gain():
    wl, params = small()
    data = I.token_batch(wl, 0)
    grad_fn = TR.make_grad_fn(wl.stage_specs, lambda t: data, wl.n_heads, wl.seq_len, wl.vocab, "f32")
    _, g0 = grad_fn(0, params, params)
    # changing backward biases, LayerNorm biases or the embedding table changes nothing
    ub = [[a.copy() for a in st] for st in params]
    ub[0][0] += 1.0                       # table
    for i, sp in enumerate(wl.stage_specs):
        ub[i][-1] += 1.0                  # Linear bias
        if sp.pre == "ln":
            ub[i][1] += 1.0               # LayerNorm bias
    _, g1 = grad_fn(0, params, ub)
    for a, b in zip(g0, g1):
        for x, y in zip(a, b):
            np.testing.assert_array_equal(x, y)
    # the first stage's backward matrix is read (the embedding needs the gradient of its output) ...
    ub = [[a.copy() for a in st] for st in params]
    ub[0][1] += 0.5
    _, g2 = grad_fn(0, params, ub)
    assert np.abs(g2[0][0] - g0[0][0]).max() > 1e-6
    np.testing.assert_array_equal(g2[0][1], g0[0][1])            # ... but never for its own weight gradient
    # a LayerNorm gain in the backward pass changes the gradients of earlier stages only
    ub = [[a.copy() for a in st] for st in params]
    ub[2][0] += 0.5                       # stage 3 = [ln, W_1]
    _, g3 = grad_fn(0, params, ub)
    np.testing.assert_array_equal(g3[2][0], g0[2][0])
    np.testing.assert_array_equal(g3[3][0], g0[3][0])
    assert np.abs(g3[1][0] - g0[1][0]).max() > 1e-8


def test_encoder_runs_through_the_recurrence_and_learns_something():
    wl = I.cfg4_small(compute="f32", steps=30)
    params0 = I.init_encoder_params(wl)
    res = TR.run_workload(wl, params0, lambda t: I.token_batch(wl, t))
    assert np.isfinite(res.losses).all()
    assert res.losses[0] == pytest.approx(np.log(wl.vocab), rel=0.15)


# ---- encoder-decoder ------------------------------------------------------------------------------------------

def small_encdec():
    wl = I.cfg5_small(compute="f32", n_enc=1, n_dec=2, d_model=8, n_heads=2, d_ff=12, seq_len=4, batch=2, vocab=11)
    params = [[a.astype(np.float64) for a in st] for st in I.init_encoder_params(wl)]
    rng = np.random.default_rng(5)
    for st in params:
        for a in st:
            a += rng.normal(size=a.shape) * 0.1
    return wl, params


def test_stage_list_and_batches_of_the_encoder_decoder():
    wl = I.cfg5()
    assert wl.n_stages == 48 + 84 + 1
    dec = wl.stage_specs[48:55]
    assert [s.post for s in dec] == ["attention", "residual", "skip_out", "cross_attention", "residual", "skip_out", "residual"]
    assert dec[0].pre == "embed_dec" and dec[0].causal and dec[2].skip_hop == 2 and dec[3].src == "memory" and dec[3].n_out == 2048
    assert wl.stage_specs[47].emit_memory and not any(s.emit_memory for s in wl.stage_specs[:47])
    assert wl.tau_fwd[0] == 2 * 132 + 1 and wl.tau_fwd[-1] == 1
    small = I.cfg5_small(vocab=50, seq_len=8, batch=4)
    src, dec_in, tgt = I.seq2seq_batch(small, 3)
    src2, _, tgt2 = I.seq2seq_batch(small, 4)
    assert src.shape == dec_in.shape == tgt.shape == (32,)
    assert (dec_in.reshape(4, 8)[:, 0] == 0).all() and (dec_in.reshape(4, 8)[:, 1:] == tgt.reshape(4, 8)[:, :-1]).all()
    # the target is one fixed permutation of the source ids, the same in every microbatch
    pi = {}
    for a, b in list(zip(src, tgt)) + list(zip(src2, tgt2)):
        assert pi.setdefault(int(a), int(b)) == int(b)
    assert len(set(pi.values())) == len(pi)
    # Zipf: rank 0 is the most frequent id
    big = I.cfg5_small(vocab=1000, seq_len=64, batch=64)
    s_big = I.seq2seq_batch(big, 0)[0]
    counts = np.bincount(s_big, minlength=1000)
    assert counts[0] == counts.max() and counts[0] > 3 * counts[10] > 0


def test_encoder_decoder_gradients_match_central_differences():
    wl, params = small_encdec()
    data = I.seq2seq_batch(wl, 0)
    grad_fn = TR.make_grad_fn(wl.stage_specs, lambda t: data, wl.n_heads, wl.seq_len, wl.vocab, "f32")
    loss, g = grad_fn(0, params, params)
    h = 1e-6
    rng = np.random.default_rng(1)
    for i, st in enumerate(params):
        for j, a in enumerate(st):
            flat = a.reshape(-1)
            for idx in rng.choice(flat.size, size=min(4, flat.size), replace=False):
                old = flat[idx]
                flat[idx] = old + h
                lp, _ = grad_fn(0, params, params)
                flat[idx] = old - h
                lm, _ = grad_fn(0, params, params)
                flat[idx] = old
                fd = (lp - lm) / (2 * h)
                assert np.asarray(g[i][j]).reshape(-1)[idx] == pytest.approx(fd, rel=3e-5, abs=3e-9), (i, j, idx)


def test_decoder_is_causal_and_reads_the_memory():
    """Changing a late decoder input token leaves the logits of earlier positions unchanged (causal self-attention,
    every other op is position-wise); changing a source token changes every position of that sequence only."""
    wl, params = small_encdec()
    src, dec_in, tgt = I.seq2seq_batch(wl, 0)
    S = wl.seq_len

    def first_stage_grad_rows(src_ids, dec_ids):
        # the loss depends on the logits only; use the per-position losses through one-hot targets
        out = []
        grad_fn = TR.make_grad_fn(wl.stage_specs, lambda t: (src_ids, dec_ids, tgt), wl.n_heads, S, wl.vocab, "f32")
        _, g = grad_fn(0, params, params)
        return g[-1][-1]                                        # bias gradient of the vocabulary projection

    def logits_of(src_ids, dec_ids):
        captured = {}
        import oracle.layers as LL
        orig = LL.cross_entropy
        def spy(logits, targets, *args):
            captured["logits"] = logits.copy()
            return orig(logits, targets, *args)
        LL.cross_entropy = spy
        try:
            TR.make_grad_fn(wl.stage_specs, lambda t: (src_ids, dec_ids, tgt), wl.n_heads, S, wl.vocab, "f32")(0, params, params)
        finally:
            LL.cross_entropy = orig
        return captured["logits"]

    base = logits_of(src, dec_in)
    d2 = dec_in.copy()
    d2[S - 1] = (d2[S - 1] + 1) % wl.vocab                      # last position of sequence 0
    changed = logits_of(src, d2)
    np.testing.assert_array_equal(changed[:S - 1], base[:S - 1])
    assert np.abs(changed[S - 1] - base[S - 1]).max() > 1e-9
    np.testing.assert_array_equal(changed[S:], base[S:])
    s2 = src.copy()
    s2[S + 1] = (s2[S + 1] + 1) % wl.vocab                      # a source token of sequence 1
    changed = logits_of(s2, dec_in)
    np.testing.assert_array_equal(changed[:S], base[:S])
    assert (np.abs(changed[S:2 * S] - base[S:2 * S]).max(axis=1) > 1e-12).all()


def test_memory_gradient_is_the_sum_over_cross_attention_stages():
    """The last encoder stage receives the sum of the gradients of every cross-attention stage: with two decoder
    layers its weight gradient differs from either single contribution, and zeroing the backward gain of one
    cross-attention stage's LayerNorm removes exactly that stage's share."""
    wl, params = small_encdec()
    data = I.seq2seq_batch(wl, 0)
    grad_fn = TR.make_grad_fn(wl.stage_specs, lambda t: data, wl.n_heads, wl.seq_len, wl.vocab, "f32")
    _, g0 = grad_fn(0, params, params)
    cross = [i for i, s in enumerate(wl.stage_specs) if s.post == "cross_attention"]
    assert len(cross) == 2
    enc_last = [i for i, s in enumerate(wl.stage_specs) if s.emit_memory][0]
    parts = []
    for keep in cross:
        ub = [[a.copy() for a in st] for st in params]
        for i in cross:
            if i != keep:
                ub[i][0][:] = 0.0                               # LayerNorm gain read in the backward pass
        _, g = grad_fn(0, params, ub)
        parts.append(g[enc_last][0])
    np.testing.assert_allclose(parts[0] + parts[1], g0[enc_last][0], rtol=1e-10, atol=1e-14)
    assert np.abs(parts[0]).max() > 1e-9 and np.abs(parts[1]).max() > 1e-9
