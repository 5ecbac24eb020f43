"""The oracle against values the paper prints (tests/golden/*.txt; each file cites its passage)."""
import math
import os

import numpy as np
import pytest

import pm_inputs as I
from oracle import recurrence as R
from oracle import update as U

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def rows(name):
    with open(os.path.join(GOLD, name)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


def test_table1_delays():
    for r in rows("table1_pipemare_delays.txt"):
        bar = r.index("|")
        P, N, fwd, bk = int(r[0]), int(r[1]), [int(x) for x in r[2:bar]], int(r[bar + 1])
        assert len(fwd) == P
        assert [math.ceil((2 * (P - i) + 1) / N) for i in range(1, P + 1)] == fwd
        if N == 1:                                   # the schedule this repository realises
            f, b = I.pipemare_delays(P)
            assert list(f) == fwd and set(b) == {bk}
    # the workloads carry exactly these delays
    assert list(I.cfg1().tau_fwd) == [7, 5, 3, 1] and list(I.cfg4().tau_fwd)[:3] == [49, 47, 45]


def test_memory_columns():
    for opt, base, pm, printed in rows("memory_columns.txt"):
        params = [np.zeros(5, dtype=np.float32)]
        state = U.fresh_opt_state(params, opt)
        # weight-sized copies the oracle's update touches: weights, gradient, optimiser moments (+ the T2 accumulator)
        copies = 1 + 1 + len(state)
        assert copies == int(base)
        assert copies + 1 == int(pm)
        assert round(int(pm) / int(base), 2) == float(printed)
        assert 0.25 <= 1.0 / int(base) <= 0.34       # 25 to 33 percent of extra weight memory


def test_figure2a_setting():
    eta = np.random.default_rng(5).normal(size=600)
    for lam, alpha, tau, diverges in rows("figure2a_setting.txt"):
        lam, alpha, tau = float(lam), float(alpha), int(tau)
        threshold = (2.0 / lam) * math.sin(math.pi / (4 * tau + 2))          # Lemma 1
        assert (alpha > threshold) == (diverges == "yes")
        params0 = [[np.array([0.0])]]

        def grad_fn(t, u_fwd, u_bkwd):
            return 0.0, [[lam * u_fwd[0][0] - eta[t]]]
        hp = dict(optimizer="sgdm", alpha=alpha, beta1=0.0, beta2=0.0, eps=0.0, t1=False, K=1, t2=False, D=0.5)
        res = R.run(params0, [tau], [tau], grad_fn, 600, hp, dtype=np.float64)
        final = abs(float(res.params[0][0][0]))
        assert (final > 1e3) == (diverges == "yes")
