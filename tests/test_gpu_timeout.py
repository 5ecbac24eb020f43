"""The failure path of the tensor-core kernels: a bounded device-side wait that expires.

No GPU is faulted or hung: the probe is a one-thread kernel without tensor memory or copies in flight whose wait
on a barrier nobody arrives at gives up after a few milliseconds, exactly as the GEMM kernels' waits would after
their one-second limit.  The library must report PM_ERR_TIMEOUT, and the context must keep working."""
import numpy as np
import pytest

import pm_inputs as I
from parity_util import run_oracle

pytestmark = pytest.mark.gpu


def test_expired_wait_is_reported_and_context_survives(cuda_device):
    import torch
    import paper_1910_05124_b200 as pm
    wl = I.cfg3_small(P=3, steps=8)
    params0 = I.init_stage_params(wl)
    teacher = I.teacher_params(wl)
    pipe = pm.Pipeline(wl, params0)
    status, message = pipe.pm_selftest_wait_timeout(4_000_000)            # about 2 ms
    assert status == "PM_ERR_TIMEOUT" and "bounded device-side wait expired" in message and "99" in message
    # the record was cleared: the same context runs a workload to the oracle's result
    P = wl.n_stages
    for s in range(wl.steps + 2 * P - 1):
        if s < wl.steps:
            x, y = I.batch(wl, s, teacher)
            pipe.pm_step(torch.from_numpy(x).cuda().to(torch.bfloat16), torch.from_numpy(y).cuda())
        else:
            pipe.pm_step(None, None)
    losses = pipe.pm_get_losses(0, wl.steps)                               # a synchronising call: would report a stale record
    res = run_oracle(wl, params0, wl.steps, teacher)
    np.testing.assert_allclose(losses, np.array(res.losses), rtol=1e-3)


def test_selftest_needs_a_tensor_core_context(cuda_device):
    import paper_1910_05124_b200 as pm
    wl = I.mlp_workload("t", 2, 64, 1, "relu", 8, compute="f32", steps=4, seed=9)
    pipe = pm.Pipeline(wl, I.init_stage_params(wl))
    status, _ = pipe.pm_selftest_wait_timeout(1000)
    assert status == "PM_ERR_UNSUPPORTED"
