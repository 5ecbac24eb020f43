"""Shared helpers of the GPU parity tests: run a workload on both sides and compare."""
import numpy as np

import pm_inputs as I


def run_gpu_pipeline(wl, params0, n_steps, teacher=None, collect_book=True, warmup=0, loop_order="tick_major"):
    """Feed n_steps microbatches through the CUDA pipeline, drain it, return (pipeline, losses, book).

    book maps (microbatch, stage 1-based) -> [forward version, backward version] as recorded by the device.
    The first `warmup` microbatches enter 2P ticks apart (synchronous warm-up), the rest one per tick.
    loop_order "mb_major": one call of pm_step per microbatch, nothing to drain.
    """
    import torch
    import paper_1910_05124_b200 as pm
    pipe = pm.Pipeline(wl, params0, loop_order=loop_order)
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
    for s in range(n_steps if mb_major else t0 + (n_steps - warmup) + 2 * P - 1):
        mb = s if mb_major else ((s // (2 * P) if s % (2 * P) == 0 else -1) if s < t0 else warmup + (s - t0))
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
                if b_mb >= 0:
                    book.setdefault((b_mb, p + 1), [None, None])[1] = b_ver
                    assert n_upd == b_ver + 1
    losses = pipe.pm_get_losses(0, n_steps)
    return pipe, losses, book


def is_encdec(wl):
    return any(sp.pre == "embed_dec" for sp in wl.stage_specs)


def run_oracle(wl, params0, n_steps, teacher=None, warmup=0):
    if wl.kind == "encoder":
        from oracle import transformer
        data = (lambda t: I.seq2seq_batch(wl, t)) if is_encdec(wl) else (lambda t: I.token_batch(wl, t))
        return transformer.run_workload(wl, params0, data, n_steps=n_steps, warmup=warmup)
    from oracle.mlp import run_workload
    teacher = I.teacher_params(wl) if teacher is None else teacher
    return run_workload(wl, params0, lambda t: I.batch(wl, t, teacher), n_steps=n_steps, warmup=warmup)


def max_rel_err(a, b):
    """max |a - b| / max |b| per tensor (the tolerance norm of the parity contract)."""
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    return float(np.abs(a - b).max() / max(np.abs(b).max(), 1e-30))


def compare_params(pipe, res, tol, per_stage=False):
    """per_stage: measure max |dw| against the largest weight of the whole stage vector (w_t)_i instead of the
    tensor's own largest entry.  Used for bf16 + Adam, where the step of an element is about alpha whatever the
    size of its gradient: an element whose gradient sign is decided by bf16 rounding noise moves by +-alpha per
    step on either side, which is large against a bias vector that is itself only a few alpha in size."""
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
                scale = max(np.abs(np.asarray(t_, dtype=np.float64)).max() for t_ in res.params[p]) if per_stage else None
                e = max_rel_err(a, ref) if scale is None else float(np.abs(a - ref).max() / scale)
                worst = max(worst, e)
                assert e <= tol, f"stage {p} tensor {j}: {e}"
        return worst
    for p, stage in enumerate(got):
        for j, (W, b) in enumerate(stage):
            eW = max_rel_err(W, res.params[p][2 * j])
            worst = max(worst, eW)
            assert eW <= tol, f"stage {p} W{j}: {eW}"
            ref_b = res.params[p][2 * j + 1]
            if np.abs(ref_b).max() > 0:
                eb = max_rel_err(b, ref_b)
                assert eb <= tol * 4, f"stage {p} b{j}: {eb}"
    return worst
