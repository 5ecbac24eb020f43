"""Pins for oracle/update.py and oracle/bf16.py: table values, hand-computed steps, library cross-checks."""
import math

import numpy as np
import pytest

from oracle import update as U
from oracle.bf16 import bf16_round


def test_t1_exponent_endpoints_and_midpoint():
    # Eq. 2: p_k = 1 - min(k/K, 1)
    assert U.t1_exponent(0, 32) == 1.0
    assert U.t1_exponent(16, 32) == 0.5
    assert U.t1_exponent(32, 32) == 0.0
    assert U.t1_exponent(1000, 32) == 0.0


def test_t1_step_size_values():
    # at k=0 the step is alpha/tau, at k>=K it is alpha, halfway it is alpha/sqrt(tau)
    assert U.t1_step_size(0.01, 7, 0, 32) == pytest.approx(0.01 / 7, rel=1e-15)
    assert U.t1_step_size(0.01, 7, 32, 32) == 0.01
    assert U.t1_step_size(0.01, 7, 16, 32) == pytest.approx(0.01 / math.sqrt(7.0), rel=1e-15)
    assert U.t1_step_size(0.01, 7, 0, 32, enabled=False) == 0.01
    # tau = 0 (synchronous stage) is not rescaled
    assert U.t1_step_size(0.01, 0, 0, 32) == 0.01


def test_t2_gamma_table():
    # gamma = D^(1/(tau_fwd - tau_bkwd)); values by independent arithmetic exp(ln D / tau)
    assert U.t2_gamma(0.5, 7, 0) == pytest.approx(math.exp(math.log(0.5) / 7), rel=1e-14)
    assert U.t2_gamma(0.5, 7, 0) == pytest.approx(0.905724, abs=5e-7)
    assert U.t2_gamma(0.1, 47, 0) == pytest.approx(0.952190, abs=5e-7)
    assert U.t2_gamma(0.1, 10, 6) == pytest.approx(0.1 ** 0.25, rel=1e-14)
    assert U.t2_gamma(0.5, 3, 3) is None


def test_gamma_theory_value_matches_D_near_exp_minus_2():
    # Appendix: gamma = 1 - 2/(tau+1) gives D = gamma^tau -> exp(-2) ~ 0.135 for large tau
    tau = 2000
    gamma = 1.0 - 2.0 / (tau + 1)
    D = gamma ** tau
    assert D == pytest.approx(math.exp(-2.0), rel=2e-3)
    assert U.t2_gamma(D, tau, 0) == pytest.approx(gamma, rel=1e-12)


def test_sgdm_hand_step():
    w, v, g = np.array([1.0]), np.array([0.5]), np.array([2.0])
    w1, v1 = U.sgdm_step(w, v, g, alpha=0.1, beta=0.9)
    assert v1[0] == pytest.approx(0.25, rel=1e-15)      # 0.9*0.5 - 0.1*2
    assert w1[0] == pytest.approx(1.25, rel=1e-15)


def test_delta_refresh_hand_step():
    d = U.delta_refresh(np.array([0.1]), np.array([1.25]), np.array([1.0]), 0.5)
    assert d[0] == pytest.approx(0.175, rel=1e-15)       # 0.5*0.1 + 0.5*0.25


def test_corrected_weights_hand_value():
    w, d = np.array([2.0, -1.0]), np.array([0.1, 0.2])
    u = U.corrected_backward_weights(w, d, 7, 0)
    np.testing.assert_allclose(u, [2.0 - 0.7, -1.0 - 1.4], rtol=1e-15)
    assert U.corrected_backward_weights(w, d, 7, 0, enabled=False) is w
    assert U.corrected_backward_weights(w, d, 3, 3) is w
    u2 = U.corrected_backward_weights(w, d, 10, 6)
    np.testing.assert_allclose(u2, [2.0 - 0.4, -1.0 - 0.8], rtol=1e-15)


def test_adam_first_step_moves_by_alpha():
    # with zero state, m_hat = g and s_hat = g^2, so the first step is alpha*g/(|g|+eps)
    g = np.array([3.0, -0.02, 1e-3])
    w = np.array([1.0, 1.0, 1.0])
    z = np.zeros(3)
    w1, m1, s1 = U.adam_step(w, z, z, g, alpha=1e-3, beta1=0.9, beta2=0.98, eps=1e-8, k=0)
    np.testing.assert_allclose(w - w1, 1e-3 * np.sign(g), rtol=2e-5)
    np.testing.assert_allclose(m1, 0.1 * g, rtol=1e-12)
    np.testing.assert_allclose(s1, 0.02 * g * g, rtol=1e-12)


def test_adam_matches_torch_adam():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(0)
    w0 = rng.normal(size=17)
    gs = rng.normal(size=(6, 17))
    p = torch.tensor(w0, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.Adam([p], lr=2e-3, betas=(0.9, 0.98), eps=1e-8)
    w, m, s = w0.copy(), np.zeros(17), np.zeros(17)
    for k in range(6):
        p.grad = torch.tensor(gs[k])
        opt.step()
        w, m, s = U.adam_step(w, m, s, gs[k], 2e-3, 0.9, 0.98, 1e-8, k)
    # torch folds the bias corrections differently (eps is added to sqrt(s)/sqrt(bc2)): same value to rounding
    np.testing.assert_allclose(w, p.detach().numpy(), rtol=1e-9, atol=1e-12)


def test_sgdm_matches_lr_inside_velocity_form_not_torch_form():
    # Appendix B.3 puts the step size inside the velocity; with a step size that changes between
    # steps this differs from the (v <- beta v + g; w <- w - alpha v) form.  Two steps by hand:
    w, v = np.array([0.0]), np.array([0.0])
    w, v = U.sgdm_step(w, v, np.array([1.0]), alpha=0.1, beta=0.5)   # v=-0.1, w=-0.1
    w, v = U.sgdm_step(w, v, np.array([1.0]), alpha=0.2, beta=0.5)   # v=-0.05-0.2=-0.25, w=-0.35
    assert w[0] == pytest.approx(-0.35, rel=1e-15)


def test_update_is_float32_when_state_is_float32():
    w = np.array([1.0], dtype=np.float32)
    st = U.fresh_opt_state(w, "sgdm")
    hp = dict(optimizer="sgdm", alpha=0.01, beta1=0.9, beta2=0.98, eps=1e-8, t1=True, K=32, t2=True, D=0.5)
    w1, st1, d1 = U.pipemare_update(w, st, np.zeros_like(w), np.array([0.3], dtype=np.float32),
                                    k=3, tau_fwd=7, tau_bkwd=0, hp=hp)
    assert w1.dtype == np.float32 and st1["v"].dtype == np.float32 and d1.dtype == np.float32
    # same step written out with explicit float32 roundings
    a = np.float32(0.01 / 7.0 ** (1.0 - 3 / 32))
    v = np.float32(np.float32(0.9) * np.float32(0)) - np.float32(a * np.float32(0.3))
    assert st1["v"][0] == np.float32(v)
    gam = np.float32(0.5 ** (1.0 / 7))
    assert d1[0] == np.float32(gam * np.float32(0)) + np.float32((np.float32(1) - gam) * np.float32(w1[0] - w[0]))


def test_tau_zero_skips_delta_and_rescale():
    hp = dict(optimizer="sgdm", alpha=0.01, beta1=0.9, beta2=0.98, eps=1e-8, t1=True, K=32, t2=True, D=0.5)
    w = np.array([1.0])
    d0 = np.array([0.0])
    w1, st1, d1 = U.pipemare_update(w, U.fresh_opt_state(w, "sgdm"), d0, np.array([1.0]),
                                    k=0, tau_fwd=0, tau_bkwd=0, hp=hp)
    assert d1 is d0
    assert w1[0] == pytest.approx(0.99, rel=1e-15)


# ---- bf16 rounding ---------------------------------------------------------------------------

def test_bf16_round_ties_to_even_bit_patterns():
    # bfloat16 keeps 8 significant bits: spacing 2^-7 just above 1
    assert bf16_round(1.0) == 1.0
    assert bf16_round(1.0 + 2.0 ** -8) == 1.0                       # tie -> even mantissa (0)
    assert bf16_round(1.0 + 3 * 2.0 ** -8) == 1.0 + 2.0 ** -6       # tie -> even mantissa (2)
    assert bf16_round(1.0 + 2.0 ** -8 + 2.0 ** -20) == 1.0 + 2.0 ** -7
    assert bf16_round(-(1.0 + 2.0 ** -8 + 2.0 ** -20)) == -(1.0 + 2.0 ** -7)
    assert bf16_round(0.0) == 0.0
    assert bf16_round(3.0e38) == pytest.approx(3.0e38, rel=2 ** -8)


def test_bf16_round_matches_torch_cast():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(1)
    x = np.concatenate([rng.normal(size=5000), rng.normal(size=5000) * 1e-6, rng.normal(size=5000) * 1e6])
    ref = torch.tensor(x, dtype=torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    np.testing.assert_array_equal(bf16_round(x), ref)
