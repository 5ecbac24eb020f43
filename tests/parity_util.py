"""Shared helpers of the GPU parity tests: run a workload on both sides and compare."""
import numpy as np

import pm_inputs as I


def run_gpu_pipeline(wl, params0, n_steps, teacher=None, collect_book=True):
    """Feed n_steps microbatches through the CUDA pipeline, drain it, return (pipeline, losses, book).

    book maps (microbatch, stage 1-based) -> [forward version, backward version] as recorded by the device.
    """
    import torch
    import paper_1910_05124_b200 as pm
    pipe = pm.Pipeline(wl, params0)
    P = len(wl.stages)
    teacher = I.teacher_params(wl) if teacher is None else teacher
    book = {}
    in_dtype = torch.bfloat16 if wl.compute == "bf16" else torch.float32
    for s in range(n_steps + 2 * P - 1):
        if s < n_steps:
            x, y = I.batch(wl, s, teacher)
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


def run_oracle(wl, params0, n_steps, teacher=None):
    from oracle.mlp import run_workload
    teacher = I.teacher_params(wl) if teacher is None else teacher
    return run_workload(wl, params0, lambda t: I.batch(wl, t, teacher), n_steps=n_steps)


def max_rel_err(a, b):
    """max |a - b| / max |b| per tensor (the tolerance norm of the parity contract)."""
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    return float(np.abs(a - b).max() / max(np.abs(b).max(), 1e-30))


def compare_params(pipe, res, tol):
    worst = 0.0
    got = pipe.unpack(pipe.w)
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
