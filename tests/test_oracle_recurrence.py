"""Pins for oracle/recurrence.py (+ quadratic.py): special cases the paper fixes and its stability theory."""
import math

import numpy as np
import pytest

from oracle import recurrence, update as U
from oracle.quadratic import quadratic_grad
from oracle.mlp import make_grad_fn


def hp_(**kw):
    hp = dict(optimizer="sgdm", alpha=0.05, beta1=0.0, beta2=0.98, eps=1e-8, t1=False, K=1, t2=False, D=0.5)
    hp.update(kw)
    return hp


def tiny_net(seed=0, P=3, d=5, T=4, act="relu"):
    rng = np.random.default_rng(seed)
    params = [[rng.normal(size=(d, d)) * 0.5, rng.normal(size=d) * 0.1] for _ in range(P)]
    X = rng.normal(size=(64, T, d))
    Y = rng.normal(size=(64, T, d))
    grad_fn = make_grad_fn([[act]] * P, lambda t: (X[t], Y[t]), "f32")
    return params, grad_fn


# ---- tau = 0: synchronous SGD, bit for bit (Section 2.1: u_fwd = u_bkwd) --------------------

@pytest.mark.parametrize("dtype", [np.float64, np.float32])
@pytest.mark.parametrize("optimizer", ["sgdm", "adam"])
def test_all_tau_zero_is_synchronous_sgd_bit_for_bit(dtype, optimizer):
    params, grad_fn = tiny_net()
    P = len(params)
    hp = hp_(optimizer=optimizer, alpha=0.03, beta1=0.9, t1=True, K=8, t2=True, D=0.5)
    res = recurrence.run(params, [0] * P, [0] * P, grad_fn, 12, hp, dtype=dtype)
    # separately written plain loop: one weight copy, ordinary gradient, ordinary optimiser
    w = [[np.array(a, dtype=dtype) for a in st] for st in params]
    st1 = [[np.zeros_like(a) for a in st] for st in w]
    st2 = [[np.zeros_like(a) for a in st] for st in w]
    losses = []
    one = dtype(1)
    for t in range(12):
        loss, g = grad_fn(t, w, w)
        losses.append(loss)
        for i in range(P):
            for j in range(2):
                gij = np.asarray(g[i][j], dtype=dtype)
                if optimizer == "sgdm":
                    st1[i][j] = dtype(0.9) * st1[i][j] - dtype(0.03) * gij
                    w[i][j] = w[i][j] + st1[i][j]
                else:
                    b1, b2 = dtype(0.9), dtype(0.98)
                    st1[i][j] = b1 * st1[i][j] + (one - b1) * gij
                    st2[i][j] = b2 * st2[i][j] + (one - b2) * (gij * gij)
                    mh = st1[i][j] / dtype(1.0 - float(b1) ** (t + 1))
                    sh = st2[i][j] / dtype(1.0 - float(b2) ** (t + 1))
                    w[i][j] = w[i][j] - (dtype(0.03) * mh) / (np.sqrt(sh) + dtype(1e-8))
    assert res.losses == losses
    for i in range(P):
        for j in range(2):
            np.testing.assert_array_equal(res.params[i][j], w[i][j])
            np.testing.assert_array_equal(res.delta[i][j], np.zeros_like(w[i][j]))


# ---- T2 off, tau_bkwd = tau_fwd: plain delayed SGD  w_{t+1} = w_t - alpha grad f_t(w_{t-tau}) ----

def test_equal_delays_is_plain_delayed_sgd_bit_for_bit():
    params, grad_fn = tiny_net(seed=3, P=3)
    tau = [5, 3, 1]
    res = recurrence.run(params, tau, tau, grad_fn, 20, hp_(alpha=0.04), dtype=np.float64)
    hist = [[[np.array(a) for a in st]] for st in params]      # hist[i][v] = version v of stage i
    for t in range(20):
        u = [hist[i][max(0, t - tau[i])] for i in range(3)]
        _, g = grad_fn(t, u, u)
        for i in range(3):
            hist[i].append([hist[i][t][j] - 0.04 * g[i][j] for j in range(2)])
    for i in range(3):
        for j in range(2):
            np.testing.assert_array_equal(res.params[i][j], hist[i][20][j])


def test_pipemare_delays_without_t2_reads_current_weights_in_backward():
    # tau_bkwd = 0, T2 off: forward version t - tau, backward version t (Section 2.2, PipeMare)
    params, grad_fn = tiny_net(seed=4, P=3)
    tau = [5, 3, 1]
    res = recurrence.run(params, tau, [0, 0, 0], grad_fn, 15, hp_(alpha=0.04), dtype=np.float64)
    hist = [[[np.array(a) for a in st]] for st in params]
    for t in range(15):
        uf = [hist[i][max(0, t - tau[i])] for i in range(3)]
        ub = [hist[i][t] for i in range(3)]
        _, g = grad_fn(t, uf, ub)
        for i in range(3):
            hist[i].append([hist[i][t][j] - 0.04 * g[i][j] for j in range(2)])
    for i in range(3):
        np.testing.assert_array_equal(res.params[i][0], hist[i][15][0])
    # and it differs from the equal-delay run (the discrepancy is real)
    res_eq = recurrence.run(params, tau, tau, grad_fn, 15, hp_(alpha=0.04), dtype=np.float64)
    assert np.abs(res_eq.params[0][0] - res.params[0][0]).max() > 1e-8


def test_bookkeeping_versions():
    params, grad_fn = tiny_net(P=3)
    tau = [5, 3, 1]
    res = recurrence.run(params, tau, [0, 0, 0], grad_fn, 9, hp_(), dtype=np.float64)
    book = {(t, i): (vf, vb) for (t, i, vf, vb) in res.book}
    assert book[(0, 1)] == (0, 0)
    assert book[(4, 1)] == (0, 4)
    assert book[(5, 1)] == (0, 5)
    assert book[(6, 1)] == (1, 6)
    assert book[(8, 2)] == (5, 8)
    assert book[(8, 3)] == (7, 8)


# ---- scalar quadratic: Lemma 1 and the characteristic polynomial of Section 3.1 -----------------

def scalar_run(tau_f, tau_b, grad_fn, n, hp, w0=1.0):
    traj = []
    recurrence.run([[np.array([w0])]], [tau_f], [tau_b], grad_fn, n, hp, dtype=np.float64,
                   on_step=lambda t, w: traj.append(float(w[0][0][0])))
    return np.array([w0] + traj)


def growth_rate(traj, lo, hi):
    """Asymptotic per-step growth factor from the envelope of |w_t| over two windows."""
    a = np.abs(traj)
    w = (hi - lo) // 2
    e1, e2 = a[lo:lo + w].max(), a[hi - w:hi].max()
    return (e2 / e1) ** (1.0 / (hi - w - lo))


@pytest.mark.parametrize("tau", [0, 1, 3, 5, 10])
def test_lemma1_threshold_is_sharp(tau):
    lam = 1.0
    a_star = (2.0 / lam) * math.sin(math.pi / (4 * tau + 2))
    n = 4000
    below = scalar_run(tau, tau, quadratic_grad(lam), n, hp_(alpha=0.97 * a_star))
    above = scalar_run(tau, tau, quadratic_grad(lam), n, hp_(alpha=1.03 * a_star))
    assert np.abs(below[-200:]).max() < 1e-3 * np.abs(below[:200]).max()
    assert np.abs(above[-200:]).max() > 1e3 * np.abs(above[:200]).max()


def test_lemma1_threshold_values():
    # (2/lambda) sin(pi/(4 tau+2)) at lambda=1: the alpha = 0.2 of Figure 2(a) is above it for tau=10 only
    vals = {t: 2.0 * math.sin(math.pi / (4 * t + 2)) for t in (0, 1, 5, 10)}
    assert vals[0] == pytest.approx(2.0) and vals[1] == pytest.approx(1.0)
    assert vals[5] > 0.2 > vals[10]


@pytest.mark.parametrize("tau,alpha", [(10, 0.2), (5, 0.2), (10, 0.1), (3, 0.3)])
def test_growth_rate_is_largest_root_of_char_poly(tau, alpha):
    # p(w) = w^(tau+1) - w^tau + alpha*lambda   (Section 3.1)
    lam = 1.0
    coeffs = np.zeros(tau + 2)
    coeffs[0], coeffs[1], coeffs[-1] = 1.0, -1.0, alpha * lam
    radius = np.abs(np.roots(coeffs)).max()
    traj = scalar_run(tau, tau, quadratic_grad(lam), 1200, hp_(alpha=alpha))
    assert growth_rate(traj, 400, 1200) == pytest.approx(radius, rel=2e-3)


def test_figure2a_setting_diverges_for_tau_10_not_for_tau_0():
    rng = np.random.default_rng(5)
    eta = rng.normal(size=600)
    big = scalar_run(10, 10, quadratic_grad(1.0, noise=lambda t: eta[t]), 600, hp_(alpha=0.2), w0=0.0)
    small = scalar_run(0, 0, quadratic_grad(1.0, noise=lambda t: eta[t]), 600, hp_(alpha=0.2), w0=0.0)
    assert np.abs(big[-50:]).max() > 1e3
    assert np.abs(small).max() < 5.0


# ---- momentum (Appendix B.3): iterate = sum_j c_j w_j^t over the roots of the momentum polynomial ----

@pytest.mark.parametrize("tau,alpha,beta", [(3, 0.02, 0.9), (7, 0.01, 0.9), (2, 0.1, 0.5)])
def test_momentum_iterates_match_mode_sum(tau, alpha, beta):
    lam, w0, n = 1.0, 1.0, 200
    traj = scalar_run(tau, tau, quadratic_grad(lam), n, hp_(alpha=alpha, beta1=beta))
    # p(w) = w^(tau+1) - (1+beta) w^tau + beta w^(tau-1) + alpha*lambda
    coeffs = np.zeros(tau + 2)
    coeffs[0], coeffs[1], coeffs[2], coeffs[-1] = 1.0, -(1 + beta), beta, coeffs[-1] + alpha * lam
    if tau == 1:
        coeffs = np.array([1.0, -(1 + beta), beta + alpha * lam])
    roots = np.roots(coeffs).astype(complex)
    # history: w_s = w0 for s = -tau..0 (zero initial velocity, clamped versions)
    ts = np.arange(-tau, 1)
    V = roots[None, :] ** ts[:, None]
    c = np.linalg.solve(V, np.full(tau + 1, w0, dtype=complex))
    pred = np.array([(c * roots ** t).sum().real for t in range(n + 1)])
    np.testing.assert_allclose(traj, pred, atol=1e-9)
    assert traj[1] == pytest.approx(w0 - alpha * lam * w0)


def test_momentum_lemma3_bound_has_unstable_alpha():
    # Lemma 3: some alpha <= (4/lambda) sin(pi/(4 tau+2)) is unstable: check the bound itself grows
    tau, beta, lam = 6, 0.9, 1.0
    a = (4.0 / lam) * math.sin(math.pi / (4 * tau + 2))
    traj = scalar_run(tau, tau, quadratic_grad(lam), 800, hp_(alpha=a, beta1=beta))
    assert np.abs(traj[-50:]).max() > 10 * np.abs(traj[:50]).max()


# ---- delay discrepancy (Section 3.2) -------------------------------------------------------------

def test_discrepancy_growth_rate_matches_its_char_poly():
    # w_{t+1} = w_t - a(l+D) w_{t-tf} + a D w_{t-tb}:  w^(tf+1) - w^tf - a D w^(tf-tb) + a(l+D)
    tf, tb, lam, Dl = 10, 6, 1.0, 5.0
    for alpha in (0.05, 0.10):
        coeffs = np.zeros(tf + 2)
        coeffs[0], coeffs[1] = 1.0, -1.0
        coeffs[(tf + 1) - (tf - tb)] += -alpha * Dl
        coeffs[-1] += alpha * (lam + Dl)
        radius = np.abs(np.roots(coeffs)).max()
        assert radius > 1.0                                        # Figure 3(a): discrepancy diverges here
        no_disc = np.zeros(tf + 2)
        no_disc[0], no_disc[1], no_disc[-1] = 1.0, -1.0, alpha * lam
        assert np.abs(np.roots(no_disc)).max() < 1.0               # ... where Delta = 0 converges
        traj = scalar_run(tf, tb, quadratic_grad(lam, Dl), 900, hp_(alpha=alpha))
        assert growth_rate(traj, 300, 900) == pytest.approx(radius, rel=2e-3)


def t2_char_poly(tf, tb, alpha, lam, Dl, gamma):
    """The T2 polynomial of the appendix, built term by term with numpy's polynomial algebra."""
    P = np.polynomial.polynomial
    w = np.array([0.0, 1.0])
    wm1, wmg = np.array([-1.0, 1.0]), np.array([-gamma, 1.0])
    wpow = lambda n: np.concatenate([np.zeros(n), [1.0]])
    p = P.polymul(P.polymul(wm1, wmg), wpow(tf))
    p = P.polyadd(p, alpha * (lam + Dl) * wmg)
    p = P.polysub(p, alpha * Dl * P.polymul(wpow(tf - tb), wmg))
    p = P.polyadd(p, alpha * Dl * (tf - tb) * (1 - gamma) * P.polymul(wpow(tf - tb), wm1))
    return p  # ascending powers


def test_t2_char_poly_construction_matches_printed_values_at_one():
    P = np.polynomial.polynomial
    tf, tb, alpha, lam, Dl, D = 10, 0, 0.05, 1.0, 5.0, 0.1
    gamma = D ** (1.0 / (tf - tb))
    p = t2_char_poly(tf, tb, alpha, lam, Dl, gamma)
    assert P.polyval(1.0, p) == pytest.approx(alpha * lam * (1 - gamma), rel=1e-10)
    assert P.polyval(1.0, P.polyder(p)) == pytest.approx(alpha * lam + 1 - gamma, rel=1e-10)


@pytest.mark.parametrize("alpha", [0.05, 0.10])
def test_t2_growth_rate_matches_t2_char_poly_for_pipemare_delays(alpha):
    tf, tb, lam, Dl, D = 10, 0, 1.0, 5.0, 0.1
    gamma = D ** (1.0 / (tf - tb))
    radius = np.abs(np.roots(t2_char_poly(tf, tb, alpha, lam, Dl, gamma)[::-1])).max()
    traj = scalar_run(tf, tb, quadratic_grad(lam, Dl), 900, hp_(alpha=alpha, t2=True, D=D))
    assert growth_rate(traj, 300, 900) == pytest.approx(radius, rel=2e-3)
    # T2 helps: without it the same setting grows faster
    traj_off = scalar_run(tf, tb, quadratic_grad(lam, Dl), 900, hp_(alpha=alpha, t2=False))
    assert growth_rate(traj_off, 300, 900) > growth_rate(traj, 300, 900)


# ---- two-weight back-propagation on the scalar chain f = (w2 w1 x - y)^2 --------------------------

def test_two_argument_gradient_on_scalar_chain():
    x, y = 0.7, -0.3
    grad_fn = make_grad_fn([["none"], ["none"]], lambda t: (np.array([[x]]), np.array([[y]])), "f32")
    z = np.zeros(1)
    uf = [[np.array([[1.5]]), z], [np.array([[-0.8]]), z]]
    ub = [[np.array([[9.0]]), z], [np.array([[0.25]]), z]]
    loss, g = grad_fn(0, uf, ub)
    r = (-0.8) * 1.5 * x - y
    assert loss == pytest.approx(r * r, rel=1e-14)
    assert g[1][0][0, 0] == pytest.approx(2 * r * 1.5 * x, rel=1e-14)        # uses only forward values
    assert g[0][0][0, 0] == pytest.approx(2 * r * 0.25 * x, rel=1e-14)       # backward value of w2
    # stage 1's backward weights are never read; the last stage's gradient ignores every u_bkwd
    ub2 = [[np.array([[-123.0]]), z], [np.array([[0.25]]), z]]
    _, g2 = grad_fn(0, uf, ub2)
    assert g2[0][0][0, 0] == g[0][0][0, 0] and g2[1][0][0, 0] == g[1][0][0, 0]


# ---- warm-up epochs (PipeMareW, Section 4): synchronous steps first, PipeMare from there -------------------------

@pytest.mark.parametrize("optimizer", ["sgdm", "adam"])
def test_warmup_covering_every_step_is_the_synchronous_run(optimizer):
    params, grad_fn = tiny_net(seed=3)
    P = len(params)
    tf, tb = [2 * (P - i) + 1 for i in range(1, P + 1)], [0] * P
    hp = hp_(optimizer=optimizer, alpha=0.03, beta1=0.9, t1=True, K=4, t2=True, D=0.5)
    warm = recurrence.run(params, tf, tb, grad_fn, 10, hp, warmup=10)
    sync = recurrence.run(params, [0] * P, [0] * P, grad_fn, 10, hp_(optimizer=optimizer, alpha=0.03, beta1=0.9))
    assert warm.losses == sync.losses
    for a, b in zip(warm.params, sync.params):
        for x, y in zip(a, b):
            np.testing.assert_array_equal(x, y)
    for st in warm.delta:
        for dlt in st:
            assert not dlt.any()                               # the accumulator is left alone during the warm-up
    assert all(vf == t and vb == t for (t, _, vf, vb) in warm.book)


def test_warmup_then_pipemare_equals_pipemare_started_from_the_warmed_weights():
    """Plain SGD keeps no optimiser state, so 'initialise with E synchronous steps' can be replayed by hand: run
    the synchronous steps, then start an ordinary PipeMare run (T1 counting from 0, delta = 0, versions clamped at
    its own start) on the remaining microbatches from those weights."""
    params, grad_fn = tiny_net(seed=4)
    P, E, n = len(params), 5, 14
    tf, tb = [2 * (P - i) + 1 for i in range(1, P + 1)], [0] * P
    hp = hp_(alpha=0.04, beta1=0.0, t1=True, K=6, t2=True, D=0.5)
    both = recurrence.run(params, tf, tb, grad_fn, n, hp, warmup=E)
    first = recurrence.run(params, [0] * P, [0] * P, grad_fn, E, hp_(alpha=0.04, beta1=0.0))
    rest = recurrence.run(first.params, tf, tb, lambda t, uf, ub: grad_fn(t + E, uf, ub), n - E, hp)
    assert both.losses == first.losses + rest.losses
    for a, b in zip(both.params, rest.params):
        for x, y in zip(a, b):
            np.testing.assert_array_equal(x, y)
    for a, b in zip(both.delta, rest.delta):
        for x, y in zip(a, b):
            np.testing.assert_array_equal(x, y)
    # versions: synchronous during the warm-up, then clamped at E while the pipeline fills
    for (t, i, vf, vb) in both.book:
        assert vb == t
        assert vf == (t if t < E else max(E, t - tf[i - 1]))


def test_warmup_keeps_adam_bias_correction_and_base_schedule_on_the_global_step():
    """One scalar parameter, gradient 1 at every step, no delays after the switch (tau = 0 everywhere), so the only
    effects of the warm-up flag are the ones under test: Adam's step is alpha_base(k) * m_hat / sqrt(s_hat) with the
    bias corrections at the global k (m_hat = s_hat = 1 for a constant gradient), hence w_k = w_0 - sum alpha_base."""
    sched = lambda k: 0.1 / (k + 1)
    hp = hp_(optimizer="adam", alpha=sched, beta1=0.9, eps=0.0, t1=True, K=3)
    res = recurrence.run([[np.array([1.0])]], [0], [0], lambda t, uf, ub: (0.0, [[np.array([1.0])]]), 9, hp,
                         dtype=np.float64, warmup=4)
    assert res.params[0][0][0] == pytest.approx(1.0 - sum(sched(k) for k in range(9)), rel=1e-12)


def test_t1_annealing_counts_from_the_switch():
    """Scalar, plain SGD, gradient 1: the step at global k >= E is alpha / tau^(1 - min((k - E)/K, 1))."""
    tau, E, K, alpha = 7, 3, 4, 0.01
    hp = hp_(alpha=alpha, t1=True, K=K)
    traj = []
    recurrence.run([[np.array([0.0])]], [tau], [0], lambda t, uf, ub: (0.0, [[np.array([1.0])]]), 10, hp,
                   dtype=np.float64, warmup=E, on_step=lambda t, w: traj.append(float(w[0][0][0])))
    steps = -np.diff([0.0] + traj)
    want = [alpha if k < E else alpha / tau ** (1.0 - min((k - E) / K, 1.0)) for k in range(10)]
    np.testing.assert_allclose(steps, want, rtol=1e-12)


# ---- N microbatches per update (Section 2.1, Table 1) -----------------------------------------------------------------

def test_n_microbatches_without_delay_equal_one_synchronous_step_on_the_whole_minibatch():
    """With every tau = 0, N microbatches of M rows whose gradients (each carrying 1/N) are accumulated and applied
    at the minibatch boundary are one synchronous step on the N*M rows: the mean loss over the minibatch is the mean
    of the microbatch means.  float64 state, so the two agree to rounding of the sum order."""
    import pm_inputs as I
    from oracle.mlp import run_workload
    N, M = 3, 8
    small = I.mlp_workload("n_micro", 3, 24, 2, "gelu", M, compute="f32", optimizer="sgdm", alpha=0.05, K=4, D=0.5, steps=4 * N, seed=123)
    small.tau_fwd = [0, 0, 0]
    big = I.mlp_workload("n_micro", 3, 24, 2, "gelu", N * M, compute="f32", optimizer="sgdm", alpha=0.05, K=4, D=0.5, steps=4, seed=123)
    big.tau_fwd = [0, 0, 0]
    params0 = I.init_stage_params(small)
    teacher = I.teacher_params(small)
    micro = lambda t: I.batch(small, t, teacher)

    def mini(u):
        xs, ys = zip(*[micro(u * N + j) for j in range(N)])
        return np.concatenate(xs), np.concatenate(ys)
    a = run_workload(small, params0, micro, n_steps=4 * N, dtype=np.float64, n_micro=N)
    b = run_workload(big, params0, mini, n_steps=4, dtype=np.float64)
    for sa, sb in zip(a.params, b.params):
        for ta, tb in zip(sa, sb):
            np.testing.assert_allclose(ta, tb, rtol=1e-11, atol=1e-14)
    # the minibatch loss is the mean of its microbatch losses
    np.testing.assert_allclose(np.array(a.losses).reshape(4, N).mean(1), np.array(b.losses), rtol=1e-12)
    # and the weights change at minibatch boundaries only
    seen = []
    run_workload(small, params0, micro, n_steps=2 * N, dtype=np.float64, n_micro=N, on_step=lambda u, w: seen.append(u))
    assert seen == [0, 1]


def test_bookkeeping_with_two_microbatches_per_update_by_hand():
    """P = 3, N = 2: Table 1 gives tau_fwd = ceil((2(P-i)+1)/N) = (3, 2, 1) updates.  Microbatches 2u and 2u+1 belong
    to update u; both read forward version max(0, u - tau_i) and backward version u."""
    import pm_inputs as I
    from oracle.mlp import run_workload
    wl = I.mlp_workload("book", 3, 8, 1, "relu", 4, compute="f32", steps=10, seed=3)
    assert I.pipemare_delays(3, 2)[0] == [3, 2, 1]
    wl.tau_fwd = I.pipemare_delays(3, 2)[0]
    res = run_workload(wl, I.init_stage_params(wl), lambda t: I.batch(wl, t), n_steps=10, n_micro=2)
    book = {(t, i): (vf, vb) for (t, i, vf, vb) in res.book}
    expect = {  # (microbatch, stage): (forward version, backward version)
        (0, 1): (0, 0), (1, 1): (0, 0), (6, 1): (0, 3), (7, 1): (0, 3), (8, 1): (1, 4), (9, 1): (1, 4),
        (4, 2): (0, 2), (5, 2): (0, 2), (6, 2): (1, 3), (9, 2): (2, 4),
        (1, 3): (0, 0), (2, 3): (0, 1), (3, 3): (0, 1), (4, 3): (1, 2), (9, 3): (3, 4)}
    for key, val in expect.items():
        assert book[key] == val, key
    assert len(res.losses) == 10


def test_accumulation_happens_in_the_state_precision_in_microbatch_order():
    """The N gradients are rounded to the state type one by one and added in order (what a gradient buffer does)."""
    from oracle import recurrence
    g = [np.array([1.0]), np.array([2.0 ** -24]), np.array([2.0 ** -24])]       # the small ones vanish against 1 in fp32
    hp = dict(optimizer="sgdm", alpha=1.0, beta1=0.0, beta2=0.0, eps=0.0, t1=False, K=1, t2=False, D=0.5)
    res = recurrence.run([[np.array([0.0])]], [0], [0], lambda t, uf, ub, loss_scale=1.0: (0.0, [[g[t]]]), 3, hp,
                         dtype=np.float32, n_micro=3)
    assert res.params[0][0][0] == np.float32(-1.0)                               # (1 + 2^-24) + 2^-24 = 1 in fp32, twice
    res64 = recurrence.run([[np.array([0.0])]], [0], [0], lambda t, uf, ub, loss_scale=1.0: (0.0, [[g[t]]]), 3, hp,
                           dtype=np.float64, n_micro=3)
    assert res64.params[0][0][0] == -(1.0 + 2.0 ** -23)


# ---- PipeMare Recompute (Appendix A.2, Appendix D) ------------------------------------------------

def recomp_char_poly(tf, tb, tr, alpha, lam, Dl, Phi, gamma):
    """The recompute polynomial of Appendix D, built term by term (ascending powers); gamma = None: no T2 correction,
    i.e. w_{t+1} = w_t - a(l+D) w_{t-tf} + a(D-Phi) w_{t-tb} + a Phi w_{t-tr} multiplied through by w^tf."""
    P = np.polynomial.polynomial
    wm1 = np.array([-1.0, 1.0])
    wpow = lambda n: np.concatenate([np.zeros(n), [1.0]])
    if gamma is None:
        p = P.polymul(wm1, wpow(tf))
        p = P.polyadd(p, [alpha * (lam + Dl)])
        p = P.polysub(p, alpha * (Dl - Phi) * wpow(tf - tb))
        return P.polysub(p, alpha * Phi * wpow(tf - tr))
    wmg = np.array([-gamma, 1.0])
    p = P.polymul(P.polymul(wm1, wmg), wpow(tf))
    p = P.polyadd(p, alpha * (lam + Dl) * wmg)
    p = P.polysub(p, alpha * (Dl - Phi) * P.polymul(wpow(tf - tb), wmg))
    p = P.polyadd(p, alpha * (Dl - Phi) * (tf - tb) * (1 - gamma) * P.polymul(wpow(tf - tb), wm1))
    p = P.polysub(p, alpha * Phi * P.polymul(wpow(tf - tr), wmg))
    p = P.polyadd(p, alpha * Phi * (tf - tr) * (1 - gamma) * P.polymul(wpow(tf - tr), wm1))
    return p


def scalar_run_recomp(tf, tb, tr, grad_fn, n, hp, w0=1.0):
    traj = []
    recurrence.run([[np.array([w0])]], [tf], [tb], grad_fn, n, hp, dtype=np.float64, tau_recomp=[tr],
                   on_step=lambda t, w: traj.append(float(w[0][0][0])))
    return np.array([w0] + traj)


def test_recompute_poly_reduces_to_the_t2_poly_when_phi_is_zero():
    tf, tb, tr, alpha, lam, Dl, D = 10, 0, 4, 0.05, 1.0, 5.0, 0.1
    gamma = D ** (1.0 / (tf - tb))
    assert np.allclose(recomp_char_poly(tf, tb, tr, alpha, lam, Dl, 0.0, gamma), t2_char_poly(tf, tb, alpha, lam, Dl, gamma))
    # and at w = 1 every delayed term cancels against the curvature: p(1) = alpha lambda (1 - gamma) for any Phi
    P = np.polynomial.polynomial
    assert P.polyval(1.0, recomp_char_poly(tf, tb, tr, alpha, lam, Dl, -5.0, gamma)) == pytest.approx(alpha * lam * (1 - gamma), rel=1e-10)


@pytest.mark.filterwarnings("ignore:overflow")
@pytest.mark.parametrize("t2", [False, True])
@pytest.mark.parametrize("alpha", [0.02, 0.05])
def test_recompute_growth_rate_matches_its_char_poly(alpha, t2):
    # the setting of the appendix's figure: Delta = 10, Phi = -5, tau_fwd = 10, tau_bkwd = 1, tau_recomp = 4, lambda = 1.
    # The polynomial is printed for the accumulator decay gamma of the pair (tau_fwd, tau_bkwd); the recurrence uses that
    # same gamma and delta for both corrections.
    tf, tb, tr, lam, Dl, Phi, D = 10, 1, 4, 1.0, 10.0, -5.0, 0.1
    gamma = D ** (1.0 / (tf - tb)) if t2 else None
    radius = np.abs(np.roots(recomp_char_poly(tf, tb, tr, alpha, lam, Dl, Phi, gamma)[::-1])).max()
    traj = scalar_run_recomp(tf, tb, tr, quadratic_grad(lam, Dl, Phi=Phi), 1200, hp_(alpha=alpha, t2=t2, D=D))
    assert growth_rate(traj, 400, 1200) == pytest.approx(radius, rel=2e-3)


def test_recompute_discrepancy_correction_widens_the_stable_range():
    # Appendix D's figure: with the correction the largest root stays below one for step sizes at which the
    # uncorrected recompute model has already left the unit circle
    tf, tb, tr, lam, Dl, Phi, D = 10, 1, 4, 1.0, 10.0, -5.0, 0.1
    gamma = D ** (1.0 / (tf - tb))
    rad = lambda a, g: np.abs(np.roots(recomp_char_poly(tf, tb, tr, a, lam, Dl, Phi, g)[::-1])).max()
    alphas = np.linspace(0.002, 0.2, 100)
    stable_plain = max(a for a in alphas if rad(a, None) < 1.0)
    stable_t2 = max(a for a in alphas if rad(a, gamma) < 1.0)
    assert stable_t2 > 1.5 * stable_plain


def test_recompute_with_the_forward_delay_changes_nothing():
    # tau_recomp = tau_fwd: the recomputation reads the forward pass's weights and the correction term has gap zero
    params, grad_plain = tiny_net(seed=4, P=4)
    rng = np.random.default_rng(4)
    X, Y = rng.normal(size=(64, 4, 5)), rng.normal(size=(64, 4, 5))
    g0 = make_grad_fn([["relu"]] * 4, lambda t: (X[t], Y[t]), "f32")
    g1 = make_grad_fn([["relu"]] * 4, lambda t: (X[t], Y[t]), "f32", segment=2)
    tf = [7, 5, 3, 1]
    hp = hp_(alpha=0.05, t2=True, D=0.3, beta1=0.9)
    a = recurrence.run(params, tf, [0] * 4, g0, 25, hp)
    b = recurrence.run(params, tf, [0] * 4, g1, 25, hp, tau_recomp=tf)
    for sa, sb in zip(a.params, b.params):
        for x, y in zip(sa, sb):
            assert np.array_equal(x, y)
    assert a.losses == b.losses


def test_recompute_gradient_by_hand_on_a_scalar_chain():
    # two scalar stages in one segment, y = w2 w1 x, loss (y - target)^2: forward with (w1f, w2f); the recomputation
    # gives stage 2 the input h' = w1r x; backward: dW2 = dy h', dh = dy w2b, dW1 = dh x, with dy from the forward's y
    x, target = 0.7, -0.3
    w1f, w2f, w1r, w2r, w1b, w2b = 1.1, -0.8, 1.3, -0.5, 0.9, -0.6
    g = make_grad_fn([["none"], ["none"]], lambda t: (np.array([[x]]), np.array([[target]])), "f32", segment=2)
    z = np.zeros(1)
    mk = lambda a, b: [[np.array([[a]]), z], [np.array([[b]]), z]]
    loss, grads = g(0, mk(w1f, w2f), mk(w1b, w2b), u_recomp=mk(w1r, w2r))
    y = w2f * w1f * x
    dy = 2 * (y - target)
    assert loss == pytest.approx((y - target) ** 2)
    assert grads[1][0][0, 0] == pytest.approx(dy * (w1r * x))
    assert grads[0][0][0, 0] == pytest.approx(dy * w2b * x)
    assert grads[1][1][0] == pytest.approx(dy) and grads[0][1][0] == pytest.approx(dy * w2b)
    # a segment boundary between the stages: stage 2 starts from the forward pass's h = w1f x
    g2 = make_grad_fn([["none"], ["none"]], lambda t: (np.array([[x]]), np.array([[target]])), "f32", segment=1)
    _, grads2 = g2(0, mk(w1f, w2f), mk(w1b, w2b), u_recomp=mk(w1r, w2r))
    assert grads2[1][0][0, 0] == pytest.approx(dy * (w1f * x))


def test_recompute_delays_follow_the_segment_pipeline():
    from oracle.mlp import recomp_delays
    P = 16
    tf = [2 * (P - i) + 1 for i in range(1, P + 1)]
    tr = recomp_delays(tf, 4)
    # Appendix A.2's example, 16 stages in 4 segments: inside a segment the j-th stage recomputes 2(S-j) steps before
    # its gradient arrives (+ 1 for the pass itself); the last segment is the forward pass itself
    assert tr == [7, 5, 3, 1] * 4
    assert tr[-4:] == tf[-4:]
    assert all(b <= a for a, b in zip(tf, tr))
    assert recomp_delays([-(-t // 2) for t in tf], 4, 2) == [4, 3, 2, 1] * 4
    # versions the recurrence reads: forward t - tau_fwd, recomputation t - tau_recomp, clamped at 0
    params, _ = tiny_net(seed=1, P=4)
    rng = np.random.default_rng(1)
    X, Y = rng.normal(size=(64, 4, 5)), rng.normal(size=(64, 4, 5))
    g = make_grad_fn([["relu"]] * 4, lambda t: (X[t], Y[t]), "f32", segment=2)
    tf4 = [7, 5, 3, 1]
    res = recurrence.run(params, tf4, [0] * 4, g, 9, hp_(), tau_recomp=recomp_delays(tf4, 2))
    assert recomp_delays(tf4, 2) == [3, 1, 3, 1]
    assert [r for r in res.book_recomp if r[0] == 8] == [(8, 1, 5), (8, 2, 7), (8, 3, 5), (8, 4, 7)]
    assert [r for r in res.book_recomp if r[0] == 2] == [(2, 1, 0), (2, 2, 1), (2, 3, 0), (2, 4, 1)]


def test_correction_reads_the_accumulator_of_the_corrected_version():
    # scalar, tau_fwd = 3, tau_recomp = 1, constant gradient 1, SGD alpha = 0.1, D = 0.5: w_t = 1 - 0.1 t,
    # gamma = 0.5^(1/3); delta_v by its recursion; u_recomp at step t is w_{t-1} - 2 delta_{t-1}
    seen = []
    def grad_fn(t, u_fwd, u_bkwd, u_recomp=None):
        seen.append(float(u_recomp[0][0][0]))
        return 0.0, [[np.array([1.0])]]
    recurrence.run([[np.array([1.0])]], [3], [0], grad_fn, 5, hp_(alpha=0.1, t2=True, D=0.5), dtype=np.float64, tau_recomp=[1])
    gamma = 0.5 ** (1.0 / 3.0)
    delta = [0.0]
    for v in range(1, 5):
        delta.append(gamma * delta[-1] + (1 - gamma) * (-0.1))
    expect = [1.0] + [(1 - 0.1 * (t - 1)) - 2 * delta[t - 1] for t in range(1, 5)]
    assert seen == pytest.approx(expect, rel=1e-12)


# ---- stage-wise stochastic delays (Appendix E) ----------------------------------------------------------------------

def test_stochastic_delays_all_zero_is_synchronous_sgd_bit_for_bit():
    params, grad_fn = tiny_net(seed=6, P=3)
    hp = hp_(alpha=0.05, beta1=0.9)
    a = recurrence.run(params, [0] * 3, [0] * 3, grad_fn, 20, hp)
    b = recurrence.run_stochastic(params, [[0] * 3] * 20, [0] * 3, grad_fn, 20, hp)
    for sa, sb in zip(a.params, b.params):
        for x, y in zip(sa, sb):
            assert np.array_equal(x, y)
    assert a.losses == b.losses


def test_stochastic_delays_constant_delay_is_delayed_sgd_on_consistent_weights():
    # one constant delay for every stage: w_{t+1} = w_t - alpha grad f_{t-tau}(w_{t-tau}), written out directly
    params, grad_fn = tiny_net(seed=7, P=3)
    tau, n, alpha = 4, 18, 0.05
    res = recurrence.run_stochastic(params, [[tau] * 3] * n, [tau] * 3, grad_fn, n, hp_(alpha=alpha), dtype=np.float64)
    w = [[np.array(a, dtype=np.float64) for a in st] for st in params]
    past = []
    for t in range(n):
        past.append(grad_fn(t, w, w)[1])
        if t - tau >= 0:
            g = past[t - tau]
            w = [[a - alpha * np.asarray(gg) for a, gg in zip(st, gs)] for st, gs in zip(w, g)]
    for sa, sb in zip(res.params, w):
        for x, y in zip(sa, sb):
            np.testing.assert_allclose(x, y, rtol=1e-13, atol=1e-15)


@pytest.mark.parametrize("tau,alpha", [(10, 0.2), (5, 0.2), (3, 0.3)])
def test_stochastic_delay_model_follows_section3_polynomial_for_a_fixed_delay(tau, alpha):
    # the gradient is taken at w_{t-tau}: on the scalar quadratic w_{t+1} = w_t - alpha lambda w_{t-tau}, whose growth rate
    # is the largest root of w^(tau+1) - w^tau + alpha lambda (Section 3)
    lam = 1.0
    traj = []
    recurrence.run_stochastic([[np.array([1.0])]], [[tau]] * 1200, [tau], quadratic_grad(lam), 1200, hp_(alpha=alpha),
                              dtype=np.float64, on_step=lambda t, w: traj.append(float(w[0][0][0])))
    coeffs = np.zeros(tau + 2)
    coeffs[0], coeffs[1], coeffs[-1] = 1.0, -1.0, alpha * lam
    assert growth_rate(np.array([1.0] + traj), 400, 1200) == pytest.approx(np.abs(np.roots(coeffs)).max(), rel=2e-3)


def test_stochastic_delays_bookkeeping_and_t1_by_hand():
    # two scalar stages, gradient 1 for both: stage 1 waits two steps, then takes steps of alpha / tau^p
    def grad_fn(t, u_fwd, u_bkwd):
        return 0.0, [[np.array([1.0])], [np.array([1.0])]]
    delays = [[2, 0], [2, 1], [2, 0], [1, 3], [0, 0]]
    hp = hp_(alpha=0.1, t1=True, K=2)
    res = recurrence.run_stochastic([[np.array([0.0])], [np.array([0.0])]], delays, [3, 1], grad_fn, 5, hp, dtype=np.float64)
    assert [b for b in res.book if b[1] == 1] == [(0, 1, -1, 0), (1, 1, -1, 0), (2, 1, 0, 1), (3, 1, 2, 2), (4, 1, 4, 3)]
    assert [b for b in res.book if b[1] == 2] == [(0, 2, 0, 1), (1, 2, 0, 2), (2, 2, 2, 3), (3, 2, 0, 4), (4, 2, 4, 5)]
    # stage 1: its k-th update (k = 0, 1, 2) uses alpha / 3^(1 - min(k/2, 1)) = 0.1/3, 0.1/sqrt(3), 0.1
    assert res.params[0][0][0] == pytest.approx(-(0.1 / 3 + 0.1 / math.sqrt(3) + 0.1), rel=1e-12)
    assert res.params[1][0][0] == pytest.approx(-0.5, rel=1e-12)
