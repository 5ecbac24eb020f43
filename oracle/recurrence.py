"""The delayed-update recurrence of Section 2.1, microbatch-major, with a queue of weight versions.

TEST INFRASTRUCTURE (see package docstring).

    w_{t+1} = w_t - alpha * grad f_t(u_fwd,t , u_bkwd,t)
    (u_fwd,t)_i  = (w_{t - tau_fwd,i})_i
    (u_bkwd,t)_i = (w_{t - tau_bkwd,i})_i  [ - (tau_fwd,i - tau_bkwd,i) * delta_{t,i}  with T2 ]

"(w_t)_i" is stage i's weights after t updates have been written to it.  The
gradient function receives both weight sets and must use u_fwd wherever the
forward pass reads a weight and u_bkwd wherever the backward pass reads one.

Readings where the paper is silent:
  * t < tau: the version index is clamped at 0 (the pipeline is still filling
    and the initial weights are the only ones that exist).
  * delta_0 = 0.
  * All reads of version t (every stage's backward) happen before any stage
    writes version t+1.
  * N microbatches per update (Section 2.1: "microbatch gradients are accumulated into gradient buffers, and weights
    are updated only at minibatch boundaries"; Table 1: tau_fwd,i = ceil((2(P-i)+1)/N), passed in by the caller):
    delays and version indices count UPDATES; microbatch t belongs to update u = t // N and every microbatch of a
    minibatch reads the same versions; the minibatch loss is the mean of its N microbatch losses, so each microbatch's
    gradient carries the factor 1/N (applied to dL/dy, where the backward pass starts) and the N gradients are added
    in microbatch order in the state precision; the update after the N-th uses step index u.  N = 1: microbatch index =
    update index.

PipeMare Recompute (Appendix A.2, Appendix D): the stages form segments of consecutive stages; only the input of a
segment's first stage is kept from the forward pass, and the activations inside a segment are computed again, just
in time for the backward pass, with the weights the stages hold by then:
    (u_recomp,t)_i = (w_{t - tau_recomp,i})_i  [ - (tau_fwd,i - tau_recomp,i) * delta_{t,i}  with T2 for recompute ]
The loss of microbatch t still comes from the forward pass (u_fwd); the backward pass takes every stashed activation
from the recomputation and reads u_bkwd as before.  Readings: tau_recomp,i is passed in by the caller; the same
accumulator and the same T2 switch serve both corrections; during a synchronous warm-up tau_recomp = 0 as well.

Which delta a correction reads: the accumulator as it stood when the corrected weights were current, i.e.
delta_{t - tau_bkwd} with w_{t - tau_bkwd} and delta_{t - tau_recomp} with w_{t - tau_recomp}.  That is what a stage
has at hand when the pass runs (updates t - tau .. t - 1 have not happened yet), and it is what the characteristic
polynomials of Section 3.2 and Appendix D encode: their correction terms carry the same power of omega as the
weights they correct.  With tau_bkwd = 0 this is delta_t, as the statement of T2 writes it.

Warm-up epochs (PipeMareW, Section 4): the first `warmup` microbatches run the synchronous baseline, i.e. the same
loop with every delay zero (standard step size, no T2 correction, delta left alone); PipeMare then starts from
those weights and optimiser state.  Readings: the pipeline is empty at the switch, so version indices are clamped
at `warmup` (the weights the warm-up produced are the only ones the filling pipeline can see); the T1 annealing
counts steps from the switch; the base step-size schedule and Adam's bias correction keep counting from 0;
delta starts at 0 at the switch.

Pins: with all tau = 0 the loop is synchronous SGD, bit for bit; with T2 off
and tau_bkwd = tau_fwd it is plain delayed SGD; on the scalar quadratic its
iterates follow the roots of the characteristic polynomials of Sections 3.1,
3.2 and Appendix B.3 (tests/test_oracle_recurrence.py).
"""
from collections import deque

import numpy as np

from . import update as U


class Result:
    def __init__(self):
        self.losses = []      # loss of microbatch t, computed from its (stale) forward weights
        self.book = []        # (t, stage index (1-based), forward version, backward version)
        self.book_recomp = [] # (t, stage index (1-based), version the recomputation read), only with tau_recomp
        self.params = None    # final per-stage lists of tensors
        self.delta = None
        self.opt = None


def run(params0, tau_fwd, tau_bkwd, grad_fn, n_steps, hp, dtype=np.float32, on_step=None, warmup=0, n_micro=1,
        tau_recomp=None):
    """Run n_steps microbatches, the first `warmup` of them synchronously; n_micro microbatches per update.

    tau_recomp: per stage, the recomputation delay (None: no recomputation); grad_fn then also receives
               u_recomp=<per-stage tensors>.

    params0:   per stage, a list of arrays (that stage's tensors).
    grad_fn:   (t, u_fwd, u_bkwd) -> (loss, grads) with grads shaped like params0.
    hp:        hyper-parameters (see update.pipemare_update).
    on_step:   optional callback (t, params) after the update of step t.
    """
    P = len(params0)
    w = [[np.array(a, dtype=dtype) for a in stage] for stage in params0]
    opt = [[U.fresh_opt_state(a, hp["optimizer"]) for a in stage] for stage in w]
    delta = [[np.zeros_like(a) for a in stage] for stage in w]
    depth = [max(tau_fwd[i], tau_bkwd[i]) + 1 for i in range(P)]
    if tau_recomp is not None:
        assert all(tau_bkwd[i] <= tau_recomp[i] <= tau_fwd[i] for i in range(P)), "tau_bkwd <= tau_recomp <= tau_fwd"
    # queue of versions per stage: hist[i][-1] is version t, hist[i][-1-d] is version t-d
    hist = [deque([w[i]], maxlen=depth[i]) for i in range(P)]
    dhist = [deque([list(delta[i])], maxlen=depth[i]) for i in range(P)]      # the accumulator next to each version
    res = Result()

    def version(i, t, lag):
        v = max(min(warmup, t), t - lag)       # nothing older than the end of the warm-up (or version 0) exists
        return v, hist[i][-1 - (t - v)], dhist[i][-1 - (t - v)]

    assert n_micro >= 1 and (n_micro == 1 or warmup == 0), "warm-up epochs are stated for one microbatch per update"
    gacc = None
    for mb in range(n_steps):
        t = mb // n_micro                       # update index: versions, delays and step counters count updates
        sync = t < warmup
        u_fwd, u_bkwd = [], []
        u_rec = None if tau_recomp is None else []
        for i in range(P):
            tf, tb = (0, 0) if sync else (tau_fwd[i], tau_bkwd[i])
            vf, wf, _ = version(i, t, tf)
            vb, wb, db = version(i, t, tb)
            u_fwd.append(wf)
            u_bkwd.append([U.corrected_backward_weights(a, d, tf, tb, hp["t2"])
                           for a, d in zip(wb, db)])
            res.book.append((mb, i + 1, vf, vb))
            if u_rec is not None:
                tr = 0 if sync else tau_recomp[i]
                vr, wr, dr = version(i, t, tr)
                # T2 for recompute (Appendix D): the same accumulator, the gap to the forward delay
                u_rec.append([U.corrected_backward_weights(a, d, tf, tr, hp["t2"]) for a, d in zip(wr, dr)])
                res.book_recomp.append((mb, i + 1, vr))
        kw = {} if n_micro == 1 else {"loss_scale": 1.0 / n_micro}
        if u_rec is not None:
            kw["u_recomp"] = u_rec
        loss, grads = grad_fn(mb, u_fwd, u_bkwd, **kw)
        res.losses.append(loss)
        g_now = [[np.asarray(g, dtype=dtype) for g in stage] for stage in grads]
        gacc = g_now if mb % n_micro == 0 else [[a + b for a, b in zip(sa, sb)] for sa, sb in zip(gacc, g_now)]
        if mb % n_micro != n_micro - 1:
            continue                            # gradients accumulate; weights change at the minibatch boundary only
        for i in range(P):
            new_stage = []
            for j, a in enumerate(w[i]):
                g = gacc[i][j]
                tf, tb = (0, 0) if sync else (tau_fwd[i], tau_bkwd[i])
                a_new, opt[i][j], delta[i][j] = U.pipemare_update(
                    a, opt[i][j], delta[i][j], g, k=t, tau_fwd=tf, tau_bkwd=tb, hp=hp, k_t1=max(t - warmup, 0))
                new_stage.append(a_new)
            w[i] = new_stage
            hist[i].append(new_stage)
            dhist[i].append(list(delta[i]))
        if on_step is not None:
            on_step(t, w)
    res.params, res.delta, res.opt = w, delta, opt
    return res


def run_stochastic(params0, delays, tau_mean, grad_fn, n_steps, hp, dtype=np.float32, on_step=None):
    """Stage-wise stochastic gradient delays (Appendix E, the Hogwild!-style variant):

        w_{i,t+1} = w_{i,t} - alpha [grad f_{t - tau_i}(w_{t - tau_i})]_i

    Every microbatch t is differentiated at ONE consistent set of weights, the current w_t (forward and backward read the
    same version), and stage i's slice of that gradient is applied tau_{i,t'} steps later: at step t stage i takes its
    slice of the gradient of microbatch t - delays[t][i].

    delays:   delays[t][i] >= 0, drawn by the caller (the appendix samples exponentials truncated at tau_max, with a
              different mean per stage).
    tau_mean: per stage, the delay the step-size rule T1 divides by (the mean of the stage's distribution, as an integer).
    Readings: while t - delays[t][i] < 0 no gradient has reached stage i yet and it is left alone (its optimiser state and
    step counters included: a stage's update index -- for the base step-size schedule, the T1 annealing and Adam's bias
    correction -- counts the updates it has applied); T2 has nothing to correct (forward and backward read the same
    weights).
    Returns a Result; book holds (t, stage (1-based), microbatch whose gradient was applied or -1, updates applied so far).
    """
    P = len(params0)
    w = [[np.array(a, dtype=dtype) for a in stage] for stage in params0]
    opt = [[U.fresh_opt_state(a, hp["optimizer"]) for a in stage] for stage in w]
    delta = [[np.zeros_like(a) for a in stage] for stage in w]
    n_applied = [0] * P
    grads_of = []                                   # grads_of[s][i]: stage i's slice of the gradient of microbatch s
    res = Result()
    hp_stage = dict(hp, t2=False)
    for t in range(n_steps):
        loss, grads = grad_fn(t, w, w)
        res.losses.append(loss)
        grads_of.append([[np.asarray(g, dtype=dtype) for g in stage] for stage in grads])
        for i in range(P):
            s = t - int(delays[t][i])
            if s < 0:
                res.book.append((t, i + 1, -1, n_applied[i]))
                continue
            new_stage = []
            for j, a in enumerate(w[i]):
                a_new, opt[i][j], delta[i][j] = U.pipemare_update(
                    a, opt[i][j], delta[i][j], grads_of[s][i][j], k=n_applied[i], tau_fwd=tau_mean[i], tau_bkwd=tau_mean[i],
                    hp=hp_stage, k_t1=n_applied[i])
                new_stage.append(a_new)
            w[i] = new_stage
            n_applied[i] += 1
            res.book.append((t, i + 1, s, n_applied[i]))
        if on_step is not None:
            on_step(t, w)
    res.params, res.delta, res.opt = w, delta, opt
    return res
