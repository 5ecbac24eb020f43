"""Pipeline of Transformer stages (encoder, or encoder-decoder) with a cross-entropy loss: grad f_t(u_fwd, u_bkwd).

TEST INFRASTRUCTURE (see package docstring).

Every stage holds exactly one weight matrix ("one stage per weight GEMM") and has the shape

    pre   : 'embed' (token embedding * sqrt(d) + sinusoidal positions; source ids)
            'embed_dec' (the same with the decoder's input ids) | 'ln' (LayerNorm) | 'none'
    linear: z = u W^T + b ;  y = act(z);  u comes from the main stream, or (src == 'memory') from the
            encoder output, which every such stage normalises with its own LayerNorm
    post  : 'attention' (split y into q, k, v; multi-head self-attention, causal if spec.causal; also hands u
                         on as a skip tensor)
            'cross_attention' (the main input is q; y is split into k, v; attention of q over k, v)
            'skip_out'  (hands u on as a skip tensor next to y)
            'residual'  (adds the skip tensor it was sent to y)
            'none'
    A skip tensor goes to the stage spec.skip_hop (default 1) positions on.  The stage with spec.emit_memory
    (the last encoder stage) also publishes its output as the memory the decoder's cross-attention stages read.

A post-LN encoder layer is four stages: [ln|embed, W_qkv, attention] [W_o, residual] [ln, W_1 + ReLU, skip_out]
[W_2, residual]; a decoder layer is seven: [ln|embed_dec, W_qkv, causal attention] [W_o, residual]
[ln, W_q, skip_out over two] [ln(memory), W_kv, cross_attention] [W_o, residual] [ln, W_1 + ReLU, skip_out]
[W_2, residual]; the last stage is [ln, W_vocab] followed by the loss.  Parameters of a stage in order:
[table] (embed), [gain, bias] (ln), W, b.

The backward pass reads u_bkwd in exactly two places (Section 2.1: the weights "used in the backward pass"):
the Linear matrix of the input-gradient product and the LayerNorm gain of dx_hat = dy * gain.  The gradients
the cross-attention stages send to the encoder output are added in descending stage order (the order in which a
pipeline produces them), each partial sum in operand precision.

Parity of whole training trajectories is unpinned by the paper; this module is pinned through finite
differences of the complete model (u_fwd = u_bkwd) and the layer-level library cross-checks.
"""
import numpy as np

from . import layers as L
from .bf16 import bf16_round


def make_grad_fn(stage_specs, data_fn, n_heads, seq_len, vocab, compute="f32", segment=None):
    """stage_specs: per stage an object with fields pre, post, act (strings).
    data_fn: t -> (ids [T] int, targets [T] int).  segment: stages per recompute segment (the gradient function
    then takes u_recomp)."""
    rnd = bf16_round if compute == "bf16" else L.identity
    f64 = lambda a: np.asarray(a, dtype=np.float64)

    def unpack(spec, tensors):
        i = 0
        out = {}
        if spec.pre in ("embed", "embed_dec"):
            out["table"] = f64(tensors[i]); i += 1
        if spec.pre == "ln":
            out["gain"], out["beta"] = f64(tensors[i]), f64(tensors[i + 1]); i += 2
        out["W"], out["b"] = f64(tensors[i]), f64(tensors[i + 1])
        return out

    def forward_range(lo, hi, weights, state, ids, dec_ids, stash):
        """Forward of stages lo..hi-1 with `weights`, starting from `state` = (main, memory, pending skip tensors);
        fills stash[i] for those stages.  Returns (state after stage hi-1, logits or None)."""
        P = len(stage_specs)
        main, memory, skip_for = state
        skip_for = dict(skip_for)
        logits = None
        for i in range(lo, hi):
            spec = stage_specs[i]
            pf = unpack(spec, weights[i])
            st = {}
            from_memory = getattr(spec, "src", "main") == "memory"
            x_in = memory if from_memory else main
            if spec.pre == "embed":
                u = L.embed_fwd(ids, pf["table"], seq_len, rnd)
            elif spec.pre == "embed_dec":
                u = L.embed_fwd(dec_ids, pf["table"], seq_len, rnd)
            elif spec.pre == "ln":
                u, st["xhat"], st["rstd"] = L.layernorm_fwd(x_in, pf["gain"], pf["beta"], rnd)
            else:
                u = x_in
            st["u"] = u
            acc = u @ rnd(pf["W"]).T + pf["b"]
            if i == P - 1:
                logits = acc                                   # fp32 on the device, not rounded
                stash[i] = st
                break
            z = rnd(acc)
            y = rnd(L.act_fwd(z, spec.act))
            st["z"] = z
            hop = getattr(spec, "skip_hop", 1)
            if spec.post == "attention":
                d = y.shape[1] // 3
                st["q"], st["k"], st["v"] = y[:, :d], y[:, d:2 * d], y[:, 2 * d:]
                main = L.attention_fwd(st["q"], st["k"], st["v"], n_heads, seq_len, getattr(spec, "causal", False), rnd)
                skip_for[i + hop] = (u, i)
            elif spec.post == "cross_attention":
                d = y.shape[1] // 2
                st["q"], st["k"], st["v"] = main, y[:, :d], y[:, d:]
                main = L.attention_fwd(st["q"], st["k"], st["v"], n_heads, seq_len, False, rnd)
            elif spec.post == "skip_out":
                main = y
                skip_for[i + hop] = (u, i)
            elif spec.post == "residual":
                sk, st["skip_src"] = skip_for.pop(i)
                main = rnd(sk + y)
            else:
                main = y
            if getattr(spec, "emit_memory", False):
                memory = main
            stash[i] = st
        return (main, memory, skip_for), logits

    def grad_fn(t, u_fwd, u_bkwd, loss_scale=1.0, u_recomp=None):
        data = data_fn(t)
        ids, targets = data[0], data[-1]
        dec_ids = data[1] if len(data) == 3 else None
        P = len(stage_specs)
        stash = [None] * P
        # the forward pass, stage by stage, keeping what every stage found on its inputs (main stream, memory,
        # skip tensors on their way): the state a recompute segment starts from
        state, state_at, logits = (None, None, {}), [], None
        for i in range(P):
            state_at.append(state)
            state, lg = forward_range(i, i + 1, u_fwd, state, ids, dec_ids, stash)
            logits = lg if lg is not None else logits
        if u_recomp is not None:
            # PipeMare Recompute (Appendix A.2): everything the backward pass reads is computed again, segment by
            # segment, from what the forward pass left at the segment's first stage (tensors that cross a segment
            # boundary -- the main input, a skip tensor, the memory -- are the forward pass's); loss and logits are not
            starts = list(range(0, P, segment))
            for a, b in zip(starts, starts[1:] + [P]):
                forward_range(a, b, u_recomp, state_at[a], ids, dec_ids, stash)

        loss, d_main = L.cross_entropy(logits, targets, rnd, loss_scale)
        d_skip_for = {}                                        # emitting stage -> gradient of the skip tensor it sent
        d_memory = None
        grads = [[None] * len(u_fwd[i]) for i in range(P)]
        for i in reversed(range(P)):
            spec, st = stage_specs[i], stash[i]
            pb = unpack(spec, u_bkwd[i])
            from_memory = getattr(spec, "src", "main") == "memory"
            if getattr(spec, "emit_memory", False):
                d_main = d_memory                              # the following stage embeds its own ids: no gradient from it
            d_prev_main = None                                 # gradient handed to the previous stage besides d_in
            if i == P - 1:
                dz = d_main                                     # dlogits, already in operand precision
            else:
                if spec.post == "attention":
                    dq, dk, dv = L.attention_bwd(d_main, st["q"], st["k"], st["v"], n_heads, seq_len,
                                                 getattr(spec, "causal", False), rnd)
                    dy = np.concatenate([dq, dk, dv], axis=1)
                elif spec.post == "cross_attention":
                    dq, dk, dv = L.attention_bwd(d_main, st["q"], st["k"], st["v"], n_heads, seq_len, False, rnd)
                    dy, d_prev_main = np.concatenate([dk, dv], axis=1), dq
                elif spec.post == "residual":
                    dy = d_main
                    d_skip_for[st["skip_src"]] = d_main
                else:
                    dy = d_main
                dz = rnd(dy * L.act_grad(st["z"], spec.act))
            dW = dz.T @ st["u"]
            db = dz.sum(axis=0)
            du = rnd(dz @ rnd(pb["W"]))
            if i in d_skip_for:
                du = du + d_skip_for.pop(i)
            g = []
            if spec.pre in ("embed", "embed_dec"):
                g.append(L.embed_bwd(du, ids if spec.pre == "embed" else dec_ids, vocab))
                d_in = None
            elif spec.pre == "ln":
                d_in, dgain, dbeta = L.layernorm_bwd(du, st["xhat"], st["rstd"], pb["gain"], rnd)
                g += [dgain, dbeta]
            else:
                d_in = du
            g += [dW, db]
            grads[i] = g
            if from_memory:
                d_memory = d_in if d_memory is None else rnd(d_memory + d_in)
                d_main = d_prev_main
            else:
                d_main = d_in
        return loss, grads

    return grad_fn


def run_workload(wl, params0, data_fn, n_steps=None, dtype=np.float32, on_step=None, warmup=0, n_micro=1, segment=None):
    """params0: per stage the list of tensors in the order [table] [gain, bias] W b.
    segment: stages per recompute segment (None: no recomputation)."""
    from . import recurrence
    from .mlp import recomp_delays
    hp = dict(optimizer=wl.optimizer, alpha=wl.alpha, beta1=wl.beta1, beta2=wl.beta2, eps=wl.eps,
              t1=wl.t1, K=wl.K, t2=wl.t2, D=wl.D)
    grad_fn = make_grad_fn(wl.stage_specs, data_fn, wl.n_heads, wl.seq_len, wl.vocab, wl.compute, segment)
    tau_recomp = None if segment is None else recomp_delays(wl.tau_fwd, segment, n_micro)
    return recurrence.run(params0, wl.tau_fwd, wl.tau_bkwd, grad_fn, wl.steps if n_steps is None else n_steps,
                          hp, dtype=dtype, on_step=on_step, warmup=warmup, n_micro=n_micro,
                          tau_recomp=tau_recomp)
