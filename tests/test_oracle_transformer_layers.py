"""Pins for the Transformer layer formulas of oracle/layers.py: library cross-checks, closed forms, finite differences."""
import numpy as np
import pytest

from oracle import layers as L

torch = pytest.importorskip("torch")
F = torch.nn.functional


def rnd_arrays(seed, *shapes):
    rng = np.random.default_rng(seed)
    return [rng.normal(size=s) for s in shapes]


def test_layernorm_forward_matches_torch_and_is_normalised():
    x, g, b = rnd_arrays(0, (7, 16), (16,), (16,))
    y, xhat, rstd = L.layernorm_fwd(x, g, b)
    ref = F.layer_norm(torch.tensor(x), (16,), torch.tensor(g), torch.tensor(b), eps=1e-5).numpy()
    np.testing.assert_allclose(y, ref, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(xhat.mean(1), 0, atol=1e-12)
    np.testing.assert_allclose((xhat ** 2).mean(1), 1, rtol=1e-4)     # biased variance, eps = 1e-5


def test_layernorm_backward_matches_autograd_and_reads_backward_gain_only_in_dx():
    x, g, b, dy = rnd_arrays(1, (5, 12), (12,), (12,), (5, 12))
    xt, gt, bt = (torch.tensor(a, requires_grad=True) for a in (x, g, b))
    F.layer_norm(xt, (12,), gt, bt, eps=1e-5).backward(torch.tensor(dy))
    _, xhat, rstd = L.layernorm_fwd(x, g, b)
    dx, dg, db = L.layernorm_bwd(dy, xhat, rstd, g)
    np.testing.assert_allclose(dx, xt.grad.numpy(), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(dg, gt.grad.numpy(), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(db, bt.grad.numpy(), rtol=1e-10, atol=1e-12)
    g2 = g + 1.0                                                       # a different backward gain
    dx2, dg2, db2 = L.layernorm_bwd(dy, xhat, rstd, g2)
    np.testing.assert_array_equal(dg2, dg)
    np.testing.assert_array_equal(db2, db)
    assert np.abs(dx2 - dx).max() > 1e-3
    # dx is linear in the backward gain: dx(g2) = dx(g) + dx(ones)
    dx1, _, _ = L.layernorm_bwd(dy, xhat, rstd, np.ones(12))
    np.testing.assert_allclose(dx2, dx + dx1, rtol=1e-10, atol=1e-12)


@pytest.mark.parametrize("causal", [False, True])
def test_attention_forward_matches_torch(causal):
    B, S, H, dk = 2, 6, 3, 4
    q, k, v = rnd_arrays(2, (B * S, H * dk), (B * S, H * dk), (B * S, H * dk))
    o = L.attention_fwd(q, k, v, H, S, causal)
    def heads(a):
        return torch.tensor(a).reshape(B, S, H, dk).permute(0, 2, 1, 3)
    ref = F.scaled_dot_product_attention(heads(q), heads(k), heads(v), is_causal=causal)
    np.testing.assert_allclose(o, ref.permute(0, 2, 1, 3).reshape(B * S, H * dk).numpy(), rtol=1e-10, atol=1e-12)


def test_attention_with_identical_keys_averages_values():
    S, H, dk = 5, 2, 3
    q, v = rnd_arrays(3, (S, H * dk), (S, H * dk))
    k = np.tile(np.random.default_rng(4).normal(size=(1, H * dk)), (S, 1))
    o = L.attention_fwd(q, k, v, H, S)
    np.testing.assert_allclose(o, np.tile(v.mean(0, keepdims=True), (S, 1)), rtol=1e-12)


@pytest.mark.parametrize("causal", [False, True])
def test_attention_backward_matches_autograd(causal):
    B, S, H, dk = 2, 5, 2, 4
    q, k, v, do = rnd_arrays(5, *[(B * S, H * dk)] * 4)
    def heads(a):
        return a.reshape(B, S, H, dk).permute(0, 2, 1, 3)
    qt, kt, vt = (torch.tensor(a, requires_grad=True) for a in (q, k, v))
    out = F.scaled_dot_product_attention(heads(qt), heads(kt), heads(vt), is_causal=causal)
    out.permute(0, 2, 1, 3).reshape(B * S, H * dk).backward(torch.tensor(do))
    dq, dk_, dv = L.attention_bwd(do, q, k, v, H, S, causal)
    np.testing.assert_allclose(dq, qt.grad.numpy(), rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(dk_, kt.grad.numpy(), rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(dv, vt.grad.numpy(), rtol=1e-9, atol=1e-11)


def test_positional_encoding_values():
    pe = L.positional_encoding(4, 8)
    assert pe[0, 0] == 0.0 and pe[0, 1] == 1.0
    assert pe[1, 0] == pytest.approx(np.sin(1.0)) and pe[1, 1] == pytest.approx(np.cos(1.0))
    assert pe[3, 2] == pytest.approx(np.sin(3.0 / 10000 ** (2 / 8)))
    assert pe[2, 7] == pytest.approx(np.cos(2.0 / 10000 ** (6 / 8)))


def test_embedding_scatter_backward_sums_repeated_tokens():
    table = np.arange(12.0).reshape(4, 3)
    ids = np.array([2, 0, 2, 1])
    dx = np.ones((4, 3))
    g = L.embed_bwd(dx, ids, 4)
    np.testing.assert_allclose(g[2], 2 * np.sqrt(3.0))          # token id 2 occurs twice
    np.testing.assert_allclose(g[3], 0.0)
    np.testing.assert_allclose(g[0], np.sqrt(3.0))


def test_embedding_forward_even_width():
    table = np.random.default_rng(6).normal(size=(5, 4))
    ids = np.array([4, 1, 1, 0, 3, 2])
    x = L.embed_fwd(ids, table, seq_len=3)
    pe = L.positional_encoding(3, 4).astype(np.float32).astype(np.float64)
    np.testing.assert_allclose(x, table[ids] * 2.0 + pe[np.arange(6) % 3], rtol=1e-15)


def test_cross_entropy_matches_torch_and_uniform_closed_form():
    logits = np.random.default_rng(7).normal(size=(6, 9)) * 3
    tg = np.array([0, 8, 3, 3, 5, 1])
    loss, dl = L.cross_entropy(logits, tg)
    lt = torch.tensor(logits, requires_grad=True)
    ref = F.cross_entropy(lt, torch.tensor(tg))
    ref.backward()
    assert loss == pytest.approx(ref.item(), rel=1e-12)
    np.testing.assert_allclose(dl, lt.grad.numpy(), rtol=1e-10, atol=1e-14)
    loss_u, dl_u = L.cross_entropy(np.zeros((4, 10)), np.array([1, 2, 3, 4]))
    assert loss_u == pytest.approx(np.log(10.0), rel=1e-14)
    np.testing.assert_allclose(dl_u.sum(axis=1), 0, atol=1e-15)


# ---- where the bf16 mode rounds (the GPU path stores or feeds bfloat16 exactly there) -----------------------------
# Each block restates the op for ONE head / one row set with the roundings written out, so that a rounding moved,
# dropped or added inside oracle/layers.py changes a bit somewhere below.

def _bf(x):
    from oracle.bf16 import bf16_round
    return bf16_round(x)


def test_bf16_rounding_points_layernorm():
    rng = np.random.default_rng(11)
    x = _bf(rng.normal(size=(5, 16)))
    g = rng.normal(size=16).astype(np.float32).astype(np.float64) + 1.0
    b = rng.normal(size=16).astype(np.float32).astype(np.float64)
    y, xhat, rstd = L.layernorm_fwd(x, g, b, _bf)
    mu = x.mean(1, keepdims=True)
    r = 1.0 / np.sqrt(((x - mu) ** 2).mean(1, keepdims=True) + 1e-5)
    np.testing.assert_array_equal(xhat, (x - mu) * r)                      # statistics and xhat stay unrounded
    np.testing.assert_array_equal(y, _bf(xhat * g + b))                    # one rounding, of the output; gain and bias in fp32
    assert np.abs(y - (xhat * g + b)).max() > 0                            # the rounding is really there
    dy = _bf(rng.normal(size=(5, 16)))
    dx, dg, db = L.layernorm_bwd(dy, xhat, rstd, g, _bf)
    np.testing.assert_array_equal(dg, (dy * xhat).sum(0))                  # parameter gradients: never rounded
    np.testing.assert_array_equal(db, dy.sum(0))
    dxh = dy * g
    ref = rstd * (dxh - dxh.mean(1, keepdims=True) - xhat * (dxh * xhat).mean(1, keepdims=True))
    np.testing.assert_array_equal(dx, _bf(ref))                            # one rounding, of dx
    assert np.abs(dx - ref).max() > 0


def test_bf16_rounding_points_attention():
    rng = np.random.default_rng(12)
    S, dk = 6, 8
    q, k, v = (_bf(rng.normal(size=(S, dk))) for _ in range(3))
    o = L.attention_fwd(q, k, v, 1, S, False, _bf)
    s = (q @ k.T) / np.sqrt(dk)
    pt = np.exp(s - s.max(1, keepdims=True))
    l = pt.sum(1, keepdims=True)                                           # row sum of the UNROUNDED exponentials
    np.testing.assert_array_equal(o, _bf((_bf(pt) @ v) / l))               # bf16(p~) feeds P.V; one rounding of O
    assert np.abs(o - _bf((_bf(pt) @ v) / _bf(pt).sum(1, keepdims=True))).max() > 0   # a rounded row sum would differ
    assert np.abs(o - _bf((pt @ v) / l)).max() > 0                         # so would an unrounded operand
    do = _bf(rng.normal(size=(S, dk)))
    dq, dkk, dv = L.attention_bwd(do, q, k, v, 1, S, False, _bf)
    p = pt / l
    np.testing.assert_array_equal(dv, _bf(_bf(p).T @ do))                  # bf16(P) as operand, result rounded
    dp = do @ v.T                                                          # dP stays unrounded
    ds = _bf(p * (dp - (dp * p).sum(1, keepdims=True)))                    # dS rounded once, as the operand of dQ and dK
    np.testing.assert_array_equal(dq, _bf((ds @ k) / np.sqrt(dk)))
    np.testing.assert_array_equal(dkk, _bf((ds.T @ q) / np.sqrt(dk)))
    ds_unr = p * (dp - (dp * p).sum(1, keepdims=True))
    assert np.abs(dq - _bf((ds_unr @ k) / np.sqrt(dk))).max() > 0          # an unrounded dS would differ
    # the causal mask removes keys after the query before the row maximum and the row sum are taken
    oc = L.attention_fwd(q, k, v, 1, S, True, _bf)
    sc = np.where(np.tril(np.ones((S, S), dtype=bool)), s, -np.inf)
    ptc = np.exp(sc - sc.max(1, keepdims=True))
    np.testing.assert_array_equal(oc, _bf((_bf(ptc) @ v) / ptc.sum(1, keepdims=True)))


def test_bf16_rounding_points_embedding_and_cross_entropy():
    rng = np.random.default_rng(13)
    V, d, S = 9, 8, 4
    table = rng.normal(size=(V, d)).astype(np.float32).astype(np.float64)
    ids = np.array([3, 0, 8, 3, 1, 1, 7, 2])
    x = L.embed_fwd(ids, table, S, _bf)
    pe = L.positional_encoding(S, d).astype(np.float32).astype(np.float64)
    ref = _bf(table)[ids] * np.sqrt(float(d)) + pe[np.arange(8) % S]       # the bf16 copy of the table is read; positions in fp32
    np.testing.assert_array_equal(x, _bf(ref))
    assert np.abs(x - _bf(table[ids] * np.sqrt(float(d)) + pe[np.arange(8) % S])).max() > 0   # the unrounded table would differ
    g = L.embed_bwd(_bf(rng.normal(size=(8, d))), ids, V)
    assert np.abs(g - _bf(g)).max() > 0                                    # the table gradient is not rounded
    logits = rng.normal(size=(5, V)) * 3
    tg = np.array([1, 0, 8, 4, 4])
    loss, dl = L.cross_entropy(logits, tg, _bf)
    m = logits.max(1, keepdims=True)
    e = np.exp(logits - m)
    sm = e / e.sum(1, keepdims=True)
    assert loss == float(np.mean(m[:, 0] + np.log(e.sum(1)) - logits[np.arange(5), tg]))   # the loss: no rounding anywhere
    sm[np.arange(5), tg] -= 1.0
    np.testing.assert_array_equal(dl, _bf(sm / 5))                         # one rounding, of the gradient
    assert np.abs(dl - sm / 5).max() > 0
