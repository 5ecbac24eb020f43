"""Pipeline of Linear+activation stages with an MSE loss: the gradient function grad f_t(u_fwd, u_bkwd).

TEST INFRASTRUCTURE (see package docstring).

A stage holds its Linear layers' tensors in the order [W_0, b_0, W_1, b_1, ...].
Forward runs stages 1..P with u_fwd; the loss is the mean squared error of the
last stage's output against the target; backward runs stages P..1 and reads
u_bkwd only in the input-gradient products (Section 2.1's two-argument
gradient).  The first layer of the network has no input gradient, so its
backward weights are never read.

Parity of whole training trajectories is unpinned by the paper; this module is
pinned through finite differences (u_fwd = u_bkwd) and through the special
cases of the recurrence that use it.
"""
import numpy as np

from . import layers as L
from .bf16 import bf16_round


def segment_starts(P, segment):
    """First stages (0-based) of the recompute segments: `segment` consecutive stages each, the last one shorter."""
    return list(range(0, P, segment))


def make_grad_fn(stage_acts, data_fn, compute="f32", segment=None):
    """stage_acts: per stage, the list of activation names of its Linear layers.
    data_fn: t -> (x [T,in], target [T,out]).  compute: 'f32' | 'bf16'.
    segment: stages per recompute segment (PipeMare Recompute, Appendix A.2); the gradient function then takes
    u_recomp and rebuilds every segment's stash from the segment's forward input with those weights."""
    rnd = bf16_round if compute == "bf16" else L.identity

    def run_stages(h, lo, hi, weights):
        """Forward of stages lo..hi-1 from input h; returns (output, [(input, z) per Linear])."""
        stash = []
        for acts, wf in zip(stage_acts[lo:hi], weights[lo:hi]):
            for j, act in enumerate(acts):
                W = np.asarray(wf[2 * j], dtype=np.float64)
                b = np.asarray(wf[2 * j + 1], dtype=np.float64)
                y, z = L.linear_fwd(h, W, b, act, rnd)
                stash.append((h, z))
                h = y
        return h, stash

    def grad_fn(t, u_fwd, u_bkwd, loss_scale=1.0, u_recomp=None):
        x, target = data_fn(t)
        P = len(stage_acts)
        h = rnd(np.asarray(x, dtype=np.float64))
        stash, stage_in = [], []
        for i in range(P):
            stage_in.append(h)
            h, st = run_stages(h, i, i + 1, u_fwd)
            stash += st
        if u_recomp is not None:
            # the loss below comes from the forward pass; what the backward pass reads is computed again per segment,
            # from the input the forward pass left at the segment's first stage
            stash = []
            starts = segment_starts(P, segment)
            for a, b in zip(starts, starts[1:] + [P]):
                stash += run_stages(stage_in[a], a, b, u_recomp)[1]
        loss, dy = L.mse_loss(h, target, rnd, loss_scale)
        grads = [[None] * len(wf) for wf in u_fwd]
        flat = len(stash) - 1
        for i in reversed(range(len(stage_acts))):
            for j in reversed(range(len(stage_acts[i]))):
                x_in, z = stash[flat]
                Wb = np.asarray(u_bkwd[i][2 * j], dtype=np.float64)
                dW, db, dy = L.linear_bwd(dy, x_in, z, Wb, stage_acts[i][j], rnd, need_dx=flat > 0)
                grads[i][2 * j], grads[i][2 * j + 1] = dW, db
                flat -= 1
        return loss, grads

    return grad_fn


def recomp_delays(tau_fwd, segment, n_micro=1):
    """tau_recomp per stage for segments of `segment` stages: inside a segment the recomputation runs ahead of the
    backward pass like the forward pass does in a pipeline of that many stages (Appendix A.2: the recomputation of the
    j-th stage of a segment of S starts 2(S-j) steps before its gradient arrives, one more step for the pass itself),
    so tau_recomp = ceil((2(S-j)+1)/N) for the j-th stage (1-based) of a segment, never above tau_fwd; the last
    segment's backward follows its forward at exactly that distance, so nothing is recomputed there
    (tau_recomp = tau_fwd)."""
    P = len(tau_fwd)
    out = []
    starts = segment_starts(P, segment)
    for a, b in zip(starts, starts[1:] + [P]):
        for i in range(a, b):
            tr = -(-(2 * (b - 1 - i) + 1) // n_micro)
            out.append(tau_fwd[i] if b == P else min(tau_fwd[i], tr))
    return out


def run_workload(wl, params0, data_fn, n_steps=None, dtype=np.float32, on_step=None, warmup=0, n_micro=1, segment=None):
    """Run a pm_inputs.Workload-like description through the recurrence.

    params0: per stage a list of (W, b) pairs.  segment: stages per recompute segment (None: no recomputation).
    Returns recurrence.Result.
    """
    from . import recurrence
    stage_acts = [[spec.act for spec in stage] for stage in wl.stages]
    flat0 = [[t for pair in stage for t in pair] for stage in params0]
    hp = dict(optimizer=wl.optimizer, alpha=wl.alpha, beta1=wl.beta1, beta2=wl.beta2, eps=wl.eps,
              t1=wl.t1, K=wl.K, t2=wl.t2, D=wl.D)
    grad_fn = make_grad_fn(stage_acts, data_fn, wl.compute, segment)
    tau_recomp = None if segment is None else recomp_delays(wl.tau_fwd, segment, n_micro)
    return recurrence.run(flat0, wl.tau_fwd, wl.tau_bkwd, grad_fn,
                          wl.steps if n_steps is None else n_steps, hp, dtype=dtype, on_step=on_step, warmup=warmup,
                          n_micro=n_micro, tau_recomp=tau_recomp)
