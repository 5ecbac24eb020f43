"""Layer formulas with separate forward and backward weight values.

TEST INFRASTRUCTURE (see package docstring).

Section 2.1 defines grad f_t(u_fwd, u_bkwd) as what back-propagation computes
when the forward pass reads u_fwd and the backward pass reads u_bkwd.  For a
Linear layer the only weight read in the backward pass is the matrix in the
input-gradient product; the weight- and bias-gradients use only stashed
forward quantities and the incoming gradient.

    forward :  z = x Wf^T + b ;  y = act(z)               stash x, z
    backward:  dz = dy * act'(z) ;  dW = dz^T x ;  db = sum_rows dz ;  dx = dz Wb

All arithmetic is float64.  `rnd` is applied wherever the bf16 GEMM path
stores a value in bfloat16 (identity for the fp32 path):
  weights as GEMM operands, the pre-activation z, the activation y, the
  incoming gradient dy, dz as GEMM operand, and the outgoing dx.
Weight- and bias-gradients are never rounded.  act and act' are evaluated at
the rounded z so that forward and backward agree on it.

GELU is the exact erf form 0.5 z (1 + erf(z / sqrt 2)).

Pins: central finite differences with u_fwd = u_bkwd (tests/test_oracle_layers.py);
the two-stage scalar chain closed form, where g_2 must not depend on u_bkwd
and g_1 = w2_bkwd * r * x.
"""
import numpy as np
from scipy.special import erf


def identity(x):
    return np.asarray(x, dtype=np.float64)


def act_fwd(z, kind):
    if kind == "relu":
        return np.maximum(z, 0.0)
    if kind == "gelu":
        return 0.5 * z * (1.0 + erf(z / np.sqrt(2.0)))
    if kind == "none":
        return z
    raise ValueError(kind)


def act_grad(z, kind):
    if kind == "relu":
        return (z > 0.0).astype(np.float64)
    if kind == "gelu":
        return 0.5 * (1.0 + erf(z / np.sqrt(2.0))) + z * np.exp(-0.5 * z * z) / np.sqrt(2.0 * np.pi)
    if kind == "none":
        return np.ones_like(z)
    raise ValueError(kind)


def linear_fwd(x, W_fwd, b_fwd, act, rnd=identity):
    """Returns (y, z).  x: [T, in], W_fwd: [out, in], b_fwd: [out]."""
    z = rnd(x @ rnd(W_fwd).T + np.asarray(b_fwd, dtype=np.float64))
    y = rnd(act_fwd(z, act))
    return y, z


def linear_bwd(dy, x, z, W_bkwd, act, rnd=identity, need_dx=True):
    """Returns (dW, db, dx).  dy: [T, out] as received (already rounded by its producer)."""
    dz = rnd(dy * act_grad(z, act))
    dW = dz.T @ x
    db = dz.sum(axis=0)
    dx = rnd(dz @ rnd(W_bkwd)) if need_dx else None
    return dW, db, dx


def mse_loss(y, target, rnd=identity):
    """loss = mean over all T*out entries of (y - target)^2 ;  dy = 2 (y - target) / (T*out)."""
    r = y - np.asarray(target, dtype=np.float64)
    loss = float(np.mean(r * r))
    dy = rnd(2.0 * r / r.size)
    return loss, dy
