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


def mse_loss(y, target, rnd=identity, grad_scale=1.0):
    """loss = mean over all T*out entries of (y - target)^2 ;  dy = grad_scale * 2 (y - target) / (T*out).
    grad_scale = 1/N when the microbatch is one of N whose mean is the minibatch loss (Section 2.1)."""
    r = y - np.asarray(target, dtype=np.float64)
    loss = float(np.mean(r * r))
    dy = rnd(2.0 * r / r.size * grad_scale)
    return loss, dy


# ---- Transformer pieces (cited architecture: post-LN encoder of "Attention is all you need") -------------
#
# Where the backward formula reads a parameter it reads the backward value (Section 2.1): the LayerNorm gain
# in dx_hat = dy * gain.  Embedding rows, positional encodings and biases are not read in the backward pass.
# LayerNorm: eps = 1e-5, biased variance.  Attention: softmax(Q K^T / sqrt(d_k)) V per head, no parameters.
# Cross-entropy: mean over tokens of logsumexp(logits) - logits[target].
#
# Rounding (`rnd`, identity for fp32): LayerNorm output; in the attention forward the P.V operand
# rnd(p~) with p~ = exp(s - rowmax) and the row sum taken from the unrounded p~, and the output O; in the
# attention backward the operands rnd(P) (for dV) and rnd(dS) (for dQ, dK) and the results dQ, dK, dV;
# residual sums; embedding output.  Statistics, logits, losses, and parameter gradients are not rounded.

LN_EPS = 1e-5


def layernorm_fwd(x, gain_fwd, bias_fwd, rnd=identity):
    """Returns (y, xhat, rstd).  x: [T, d]."""
    mu = x.mean(axis=1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=1, keepdims=True)
    rstd = 1.0 / np.sqrt(var + LN_EPS)
    xhat = (x - mu) * rstd
    y = rnd(xhat * np.asarray(gain_fwd, dtype=np.float64) + np.asarray(bias_fwd, dtype=np.float64))
    return y, xhat, rstd


def layernorm_bwd(dy, xhat, rstd, gain_bkwd, rnd=identity):
    """Returns (dx, dgain, dbias).  dgain/dbias use only stashed forward quantities."""
    dgain = (dy * xhat).sum(axis=0)
    dbias = dy.sum(axis=0)
    dxhat = dy * np.asarray(gain_bkwd, dtype=np.float64)
    dx = rstd * (dxhat - dxhat.mean(axis=1, keepdims=True) - xhat * (dxhat * xhat).mean(axis=1, keepdims=True))
    return rnd(dx), dgain, dbias


def attention_fwd(q, k, v, n_heads, seq_len, causal=False, rnd=identity):
    """q, k, v: [T, d] with T = batch * seq_len, heads are contiguous slices of d.  Returns o [T, d]."""
    T, d = q.shape
    dk = d // n_heads
    B = T // seq_len
    o = np.zeros((T, d))
    scale = 1.0 / np.sqrt(dk)
    for b in range(B):
        rows = slice(b * seq_len, (b + 1) * seq_len)
        for h in range(n_heads):
            cols = slice(h * dk, (h + 1) * dk)
            s = (q[rows, cols] @ k[rows, cols].T) * scale
            if causal:
                s = np.where(np.tril(np.ones((seq_len, seq_len), dtype=bool)), s, -np.inf)
            p = np.exp(s - s.max(axis=1, keepdims=True))
            l = p.sum(axis=1, keepdims=True)
            o[rows, cols] = (rnd(p) @ v[rows, cols]) / l
    return rnd(o)


def attention_bwd(do, q, k, v, n_heads, seq_len, causal=False, rnd=identity):
    """Returns (dq, dk, dv).  P is recomputed from q, k exactly as in the forward pass."""
    T, d = q.shape
    dk_ = d // n_heads
    B = T // seq_len
    dq, dkk, dv = np.zeros((T, d)), np.zeros((T, d)), np.zeros((T, d))
    scale = 1.0 / np.sqrt(dk_)
    for b in range(B):
        rows = slice(b * seq_len, (b + 1) * seq_len)
        for h in range(n_heads):
            cols = slice(h * dk_, (h + 1) * dk_)
            s = (q[rows, cols] @ k[rows, cols].T) * scale
            if causal:
                s = np.where(np.tril(np.ones((seq_len, seq_len), dtype=bool)), s, -np.inf)
            pt = np.exp(s - s.max(axis=1, keepdims=True))
            l = pt.sum(axis=1, keepdims=True)
            p = pt / l                                   # softmax
            dO = do[rows, cols]
            dv[rows, cols] = rnd(p).T @ dO               # P as a matrix-product operand
            dp = dO @ v[rows, cols].T
            ds = p * (dp - (dp * p).sum(axis=1, keepdims=True))
            ds = rnd(ds)
            dq[rows, cols] = (ds @ k[rows, cols]) * scale
            dkk[rows, cols] = (ds.T @ q[rows, cols]) * scale
    return rnd(dq), rnd(dkk), rnd(dv)


def positional_encoding(seq_len, d):
    """Sinusoidal positions: PE[pos, 2i] = sin(pos / 10000^(2i/d)), PE[pos, 2i+1] = cos(same)."""
    pos = np.arange(seq_len)[:, None].astype(np.float64)
    i = np.arange(d // 2)[None, :].astype(np.float64)
    ang = pos / np.power(10000.0, 2.0 * i / d)
    pe = np.zeros((seq_len, d))
    pe[:, 0::2] = np.sin(ang)
    pe[:, 1::2] = np.cos(ang)
    return pe


def embed_fwd(ids, table_fwd, seq_len, rnd=identity):
    """x = table[ids] * sqrt(d) + PE[position].  ids: [T] with T = batch * seq_len."""
    d = table_fwd.shape[1]
    pe = positional_encoding(seq_len, d).astype(np.float32).astype(np.float64)   # held in fp32 on the device
    pos = np.arange(ids.shape[0]) % seq_len
    return rnd(rnd(table_fwd)[ids] * np.sqrt(float(d)) + pe[pos])


def embed_bwd(dx, ids, vocab):
    """dTable[ids[t]] += dx[t] * sqrt(d), tokens in ascending order."""
    d = dx.shape[1]
    g = np.zeros((vocab, d))
    np.add.at(g, ids, dx * np.sqrt(float(d)))
    return g


def cross_entropy(logits, targets, rnd=identity, grad_scale=1.0):
    """loss = mean_t (logsumexp(logits_t) - logits_t[target_t]);  dlogits = grad_scale * (softmax - onehot) / T."""
    T = logits.shape[0]
    m = logits.max(axis=1, keepdims=True)
    e = np.exp(logits - m)
    ssum = e.sum(axis=1, keepdims=True)
    lse = m[:, 0] + np.log(ssum[:, 0])
    loss = float(np.mean(lse - logits[np.arange(T), targets]))
    dl = e / ssum
    dl[np.arange(T), targets] -= 1.0
    return loss, rnd(dl / T * grad_scale)
