"""Shared helpers of the GPU parity tests: run a workload on both sides and compare."""
import numpy as np

import pm_inputs as I


def run_gpu_pipeline(wl, params0, n_steps, teacher=None, collect_book=True, warmup=0, loop_order="tick_major", n_micro=1, entry_period=1,
                     segment=0, book_recomp=None, fuse_update=0, delays=None, tau_max=0, book_applied=None, materialize=0):
    """Feed n_steps microbatches through the CUDA pipeline, drain it, return (pipeline, losses, book).

    book maps (microbatch, stage 1-based) -> [forward version, backward version] as recorded by the device.
    The first `warmup` microbatches enter 2P ticks apart (synchronous warm-up), the rest one per tick.
    loop_order "mb_major": one call of pm_step per microbatch, nothing to drain.
    segment: stages per recompute segment (PipeMare Recompute); book_recomp, a dict, then receives
    (microbatch, stage 1-based) -> version the recomputation read.
    delays, tau_max: the stage-wise stochastic delay model: delays[t][i] is set before step t; book_applied, a dict, then
    receives (step, stage 1-based) -> (microbatch whose gradient was applied or -1, updates applied after the step).
    """
    import torch
    import paper_1910_05124_b200 as pm
    pipe = pm.Pipeline(wl, params0, loop_order=loop_order, n_micro=n_micro, entry_period=entry_period, recompute_segment=segment,
                       fuse_update=fuse_update, stochastic_tau_max=tau_max, materialize_backward=materialize)
    P = wl.n_stages
    encoder = wl.kind == "encoder"
    if not encoder:
        teacher = I.teacher_params(wl) if teacher is None else teacher
    book = {}
    in_dtype = torch.bfloat16 if wl.compute == "bf16" else torch.float32
    warmup = min(warmup, n_steps)
    if warmup:
        pipe.pm_set_warmup(warmup)
    t0 = 2 * P * warmup                                        # first tick of the one-per-tick phase
    mb_major = pipe.mb_major
    E = entry_period                                            # tick-major: a microbatch enters every E ticks
    n_ticks = n_steps if mb_major else ((n_steps - 1) * E + 2 * P if E > 1 else t0 + (n_steps - warmup) + 2 * P - 1)
    for s in range(n_ticks):
        if mb_major:
            mb = s
        elif E > 1:
            mb = s // E if s % E == 0 else -1
        else:
            mb = (s // (2 * P) if s % (2 * P) == 0 else -1) if s < t0 else warmup + (s - t0)
        if delays is not None:
            pipe.pm_set_delays(delays[s])
        if 0 <= mb < n_steps:
            if encoder and is_encdec(wl):
                src, dec_in, tg = I.seq2seq_batch(wl, mb)              # two token streams: [source | decoder input]
                xd = torch.from_numpy(np.concatenate([src, dec_in]).astype(np.int32)).to(pipe.device)
                yd = torch.from_numpy(tg.astype(np.int32)).to(pipe.device)
            elif encoder:
                ids, tg = I.token_batch(wl, mb)
                xd = torch.from_numpy(ids.astype(np.int32)).to(pipe.device)
                yd = torch.from_numpy(tg.astype(np.int32)).to(pipe.device)
            else:
                x, y = I.batch(wl, mb, teacher)
                xd = torch.from_numpy(x).to(pipe.device).to(in_dtype)
                yd = torch.from_numpy(y).to(pipe.device)
            pipe.pm_step(xd, yd)
        else:
            pipe.pm_step(None, None)
        if collect_book:
            for p in range(P):
                f_mb, f_ver, b_mb, b_ver, n_upd, f_slot, b_slot, tick = pipe.pm_get_bookkeeping(p)
                assert tick == s
                if f_mb >= 0:
                    book.setdefault((f_mb, p + 1), [None, None])[0] = f_ver
                if book_applied is not None:
                    book_applied[(s, p + 1)] = (b_slot, n_upd)
                    continue
                if b_mb >= 0:
                    book.setdefault((b_mb, p + 1), [None, None])[1] = b_ver
                    assert n_upd == b_ver + (1 if (b_mb + 1) % n_micro == 0 else 0)      # the update follows the N-th microbatch
                    if book_recomp is not None:
                        book_recomp[(b_mb, p + 1)] = b_slot                              # with recompute: the version it read
    losses = pipe.pm_get_losses(0, n_steps)
    return pipe, losses, book


def is_encdec(wl):
    return any(sp.pre == "embed_dec" for sp in wl.stage_specs)


def run_oracle(wl, params0, n_steps, teacher=None, warmup=0, n_micro=1, segment=None):
    if wl.kind == "encoder":
        from oracle import transformer
        data = (lambda t: I.seq2seq_batch(wl, t)) if is_encdec(wl) else (lambda t: I.token_batch(wl, t))
        return transformer.run_workload(wl, params0, data, n_steps=n_steps, warmup=warmup, n_micro=n_micro, segment=segment)
    from oracle.mlp import run_workload
    teacher = I.teacher_params(wl) if teacher is None else teacher
    return run_workload(wl, params0, lambda t: I.batch(wl, t, teacher), n_steps=n_steps, warmup=warmup, n_micro=n_micro, segment=segment)


def max_rel_err(a, b):
    """max |a - b| / max |b| per tensor (the tolerance norm of the parity contract)."""
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    return float(np.abs(a - b).max() / max(np.abs(b).max(), 1e-30))


def compare_params(pipe, res, tol, per_stage=False, bias_per_stage=False, report=None):
    """per_stage: measure max |dw| against the largest weight of the whole stage vector (w_t)_i instead of the
    tensor's own largest entry.  Used for bf16 + Adam, where the step of an element is about alpha whatever the
    size of its gradient: an element whose gradient sign is decided by bf16 rounding noise moves by +-alpha per
    step on either side, which is large against a bias vector that is itself only a few alpha in size.
    bias_per_stage: the stage norm for bias vectors only (Linear and LayerNorm biases: the tensors that are a few alpha
    in size); weight matrices, embedding tables and LayerNorm gains are held to their own largest entry.
    report: optional dict that receives the worst per-tensor and per-stage-vector errors, whichever is asserted."""
    worst = 0.0
    got = pipe.unpack(pipe.w)
    if pipe.is_encoder:
        wl = pipe.wl
        for p, stage in enumerate(got):
            sp = wl.stage_specs[p]
            for j, a in enumerate(stage):
                ref = np.asarray(res.params[p][j], dtype=np.float64)
                a = np.asarray(a, dtype=np.float64)
                if sp.post == "attention" and j == len(stage) - 1:
                    # The key bias is a gauge direction: softmax(q k^T) does not depend on it, its exact
                    # gradient is zero, and what reaches the optimiser is rounding noise (which Adam turns into
                    # steps of up to alpha).  It is checked against that bound instead of element by element.
                    d = sp.n_out // 3
                    bound = wl.alpha * len(res.losses) * 1.01 + 1e-12
                    assert np.abs(a[d:2 * d]).max() <= bound and np.abs(ref[d:2 * d]).max() <= bound
                    keep = np.r_[0:d, 2 * d:3 * d]
                    a, ref = a[keep], ref[keep]
                if sp.post == "cross_attention" and j == len(stage) - 1:
                    d = sp.n_out // 2                            # [k | v]: the same gauge direction, first half
                    bound = wl.alpha * len(res.losses) * 1.01 + 1e-12
                    assert np.abs(a[:d]).max() <= bound and np.abs(ref[:d]).max() <= bound
                    a, ref = a[d:], ref[d:]
                stage_scale = max(np.abs(np.asarray(t_, dtype=np.float64)).max() for t_ in res.params[p])
                e_tensor, e_stage = max_rel_err(a, ref), float(np.abs(a - ref).max() / stage_scale)
                n_t = len(stage)
                is_bias = j == n_t - 1 or (sp.pre == "ln" and j == 1)          # Linear bias (last tensor), LayerNorm bias
                use_stage = per_stage or (bias_per_stage and is_bias)
                e = e_stage if use_stage else e_tensor
                if report is not None:
                    report["per_tensor"] = max(report.get("per_tensor", 0.0), e_tensor)
                    report["per_stage_vector"] = max(report.get("per_stage_vector", 0.0), e_stage)
                    if not is_bias:
                        report["per_tensor_without_biases"] = max(report.get("per_tensor_without_biases", 0.0), e_tensor)
                worst = max(worst, e)
                assert e <= tol, f"stage {p} tensor {j}: {e} (per tensor {e_tensor}, per stage vector {e_stage})"
        return worst
    for p, stage in enumerate(got):
        for j, (W, b) in enumerate(stage):
            eW = max_rel_err(W, res.params[p][2 * j])
            worst = max(worst, eW)
            assert eW <= tol, f"stage {p} W{j}: {eW}"
            ref_b = res.params[p][2 * j + 1]
            if np.abs(ref_b).max() > 0:
                # a bias starts at zero and is a few steps in size: it is held to the tolerance against the largest entry
                # of its stage vector (w_t)_i, the unit in which Section 2.1 states the method, not against itself
                stage_scale = max(np.abs(np.asarray(t_, dtype=np.float64)).max() for t_ in res.params[p])
                eb = float(np.abs(np.asarray(b, dtype=np.float64) - np.asarray(ref_b, dtype=np.float64)).max() / stage_scale)
                worst = max(worst, eb)
                assert eb <= tol, f"stage {p} b{j}: {eb} of the stage vector's largest entry"
    return worst


def adam_tensor_stats(a, ref, alpha, n_updates, tol=2e-2):
    """Error measures of one tensor under bf16 + Adam.  Adam's step of an element is about alpha whatever the size of
    its gradient, so an element whose gradient is rounding noise walks +-alpha per update on either side and the
    max-norm of the difference is bounded by 2 alpha n_updates, not by the operand precision; what the operand
    precision does bound is the bulk of the elements.  Returns (relative L2 error, fraction of elements beyond
    tol * max|ref|, max |difference| / (2 alpha n_updates))."""
    a = np.asarray(a, dtype=np.float64).ravel()
    ref = np.asarray(ref, dtype=np.float64).ravel()
    d = np.abs(a - ref)
    l2 = float(np.sqrt((d * d).sum()) / max(np.sqrt((ref * ref).sum()), 1e-30))
    frac = float((d > tol * max(np.abs(ref).max(), 1e-30)).mean())
    return l2, frac, float(d.max() / (2.0 * alpha * n_updates))


def compare_params_adam(pipe, res, n_updates, tol=2e-2, max_frac=0.01, report=None):
    """bf16 + Adam over many updates, per tensor: relative L2 error <= tol; at most max_frac of the elements further
    than tol * max|w| from the oracle; no element further than the two-sided Adam walk 2 alpha n_updates.
    Bias vectors (Linear and LayerNorm biases), which are themselves only a few alpha in size, are measured against
    the largest entry of their stage vector (w_t)_i instead of their own, and their L2 error against the stage's.
    The key-bias gauge direction of attention stages is bounded by alpha n_updates as in compare_params."""
    wl = pipe.wl
    got = pipe.unpack(pipe.w)
    worst = {"l2": 0.0, "frac_beyond_tol": 0.0, "max_over_adam_walk": 0.0}
    bad = []
    for p, stage in enumerate(got):
        sp = wl.stage_specs[p]
        stage_max = max(np.abs(np.asarray(t_, dtype=np.float64)).max() for t_ in res.params[p])
        stage_l2 = np.sqrt(sum(float((np.asarray(t_, dtype=np.float64) ** 2).sum()) for t_ in res.params[p]))
        for j, a in enumerate(stage):
            ref = np.asarray(res.params[p][j], dtype=np.float64)
            a = np.asarray(a, dtype=np.float64)
            is_bias = j == len(stage) - 1 or (sp.pre == "ln" and j == 1)
            if sp.post in ("attention", "cross_attention") and j == len(stage) - 1:
                d = sp.n_out // (3 if sp.post == "attention" else 2)
                lo = d if sp.post == "attention" else 0
                bound = wl.alpha * n_updates * 1.01 + 1e-12
                assert np.abs(a[lo:lo + d]).max() <= bound and np.abs(ref[lo:lo + d]).max() <= bound
                keep = np.r_[0:lo, lo + d:a.shape[0]]
                a, ref = a[keep], ref[keep]
            diff = np.abs(a - ref).ravel()
            walk = float(diff.max() / (2.0 * wl.alpha * n_updates))
            scale = stage_max if is_bias else max(np.abs(ref).max(), 1e-30)
            l2 = float(np.sqrt((diff * diff).sum()) / (stage_l2 if is_bias else max(np.sqrt((ref * ref).sum()), 1e-30)))
            frac = float((diff > tol * scale).mean())
            worst["l2"] = max(worst["l2"], l2)
            worst["frac_beyond_tol"] = max(worst["frac_beyond_tol"], frac)
            worst["max_over_adam_walk"] = max(worst["max_over_adam_walk"], walk)
            if l2 > tol or frac > max_frac or walk > 1.0:
                bad.append(f"stage {p} tensor {j}{' (bias)' if is_bias else ''}: L2 {l2:.3g}, beyond tol {frac:.3g}, of the Adam walk {walk:.3g}")
    if report is not None:
        report.update(worst)
    assert not bad, "; ".join(bad)
    return worst
