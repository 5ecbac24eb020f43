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
