"""Finite-difference pins for oracle/layers.py and oracle/mlp.py (u_fwd = u_bkwd, no rounding)."""
import numpy as np
import pytest

from oracle import layers as L
from oracle.mlp import make_grad_fn


@pytest.mark.parametrize("act", ["relu", "gelu", "none"])
@pytest.mark.parametrize("per_stage", [1, 2])
def test_mlp_gradients_match_central_differences(act, per_stage):
    rng = np.random.default_rng(7)
    P, T = 3, 4
    dims = [5, 6, 4, 7, 3, 5, 6][: P * per_stage + 1]
    params, acts, k = [], [], 0
    for i in range(P):
        st, a = [], []
        for j in range(per_stage):
            st += [rng.normal(size=(dims[k + 1], dims[k])) * 0.6, rng.normal(size=dims[k + 1]) * 0.3]
            a.append(act)
            k += 1
        params.append(st)
        acts.append(a)
    x = rng.normal(size=(T, dims[0]))
    y = rng.normal(size=(T, dims[k]))
    grad_fn = make_grad_fn(acts, lambda t: (x, y), "f32")
    loss, g = grad_fn(0, params, params)
    h = 1e-6
    for i in range(P):
        for j, a in enumerate(params[i]):
            it = np.nditer(a, flags=["multi_index"])
            checked = 0
            for _ in it:
                idx = it.multi_index
                if checked >= 12:
                    break
                old = a[idx]
                a[idx] = old + h
                lp, _ = grad_fn(0, params, params)
                a[idx] = old - h
                lm, _ = grad_fn(0, params, params)
                a[idx] = old
                fd = (lp - lm) / (2 * h)
                assert g[i][j][idx] == pytest.approx(fd, rel=2e-5, abs=1e-9)
                checked += 1


def test_gelu_values_and_derivative():
    # GELU(0)=0, GELU'(0)=1/2, GELU(z)->z for large z; derivative by central difference
    assert L.act_fwd(np.array([0.0]), "gelu")[0] == 0.0
    assert L.act_grad(np.array([0.0]), "gelu")[0] == pytest.approx(0.5)
    assert L.act_fwd(np.array([10.0]), "gelu")[0] == pytest.approx(10.0, rel=1e-12)
    z = np.linspace(-4, 4, 41)
    h = 1e-6
    fd = (L.act_fwd(z + h, "gelu") - L.act_fwd(z - h, "gelu")) / (2 * h)
    np.testing.assert_allclose(L.act_grad(z, "gelu"), fd, rtol=1e-7, atol=1e-9)
    # Phi(1) = 0.8413447460685429 (standard normal CDF), GELU(1) = Phi(1)
    assert L.act_fwd(np.array([1.0]), "gelu")[0] == pytest.approx(0.8413447460685429, rel=1e-12)


def test_mse_definition():
    y = np.array([[1.0, 2.0], [3.0, 5.0]])
    t = np.array([[0.0, 2.0], [1.0, 1.0]])
    loss, dy = L.mse_loss(y, t)
    assert loss == pytest.approx((1 + 0 + 4 + 16) / 4)
    np.testing.assert_allclose(dy, 2 * (y - t) / 4)


def test_bf16_mode_rounds_at_stated_points():
    from oracle.bf16 import bf16_round
    rng = np.random.default_rng(2)
    x = bf16_round(rng.normal(size=(3, 8)))
    W = rng.normal(size=(4, 8)).astype(np.float32).astype(np.float64)
    b = rng.normal(size=4).astype(np.float32).astype(np.float64)
    y, z = L.linear_fwd(x, W, b, "gelu", bf16_round)
    np.testing.assert_array_equal(z, bf16_round(x @ bf16_round(W).T + b))
    np.testing.assert_array_equal(y, bf16_round(L.act_fwd(z, "gelu")))
    dy = bf16_round(rng.normal(size=(3, 4)))
    dW, db, dx = L.linear_bwd(dy, x, z, W, "gelu", bf16_round)
    dz = bf16_round(dy * L.act_grad(z, "gelu"))
    np.testing.assert_array_equal(dW, dz.T @ x)          # not rounded
    np.testing.assert_array_equal(db, dz.sum(0))
    np.testing.assert_array_equal(dx, bf16_round(dz @ bf16_round(W)))
