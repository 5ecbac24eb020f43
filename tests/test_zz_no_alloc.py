"""pm_update_flat_static: the fused update for callers that cannot allocate device memory.

A host that lives under someone else's allocator (a framework's caching pool, a real-time loop with
allocation switched off after start-up, a plug-in handed tensors only) cannot give pm_update_flat the
device workspace it wants.  The static variant keeps that table in a fixed array inside the library.
This file checks, through the C ABI, that it produces the same bits as pm_update_flat on two calls in
a row (the array is shared and keeps the previous call's contents, so the second call must not be
disturbed by the first), and that it refuses more stages than the array was sized for.

The file name sorts last so that a run that stops at the first failure has already run every other test.
"""
import numpy as np
import pytest

import pm_inputs as I

pytestmark = pytest.mark.gpu


def run_two_calls(case, optimizer, static, stream=None, check_no_alloc=False):
    import torch
    import paper_1910_05124_b200 as pm
    dev = torch.device("cuda:0")
    t = {n: torch.from_numpy(case[n]).to(dev) for n in ("w", "m", "delta", "g")}
    s = torch.from_numpy(case["s"]).to(dev) if optimizer == "adam" else None
    lp = torch.zeros(case["total"], dtype=torch.bfloat16, device=dev)
    fu = pm.FlatUpdate(case["offsets"], case["counts"], case["tau_fwd"], case["tau_bkwd"], optimizer=optimizer,
                       alpha=0.01 if optimizer == "sgdm" else 5e-4, K=32, D=0.5)
    call = fu.pm_update_flat_static if static else fu.pm_update_flat
    snaps = []
    if static and check_no_alloc:
        call(t["w"], t["m"], s, t["delta"], t["g"], lp, 8)          # the first call on a device looks up the array's address
        torch.cuda.synchronize()
        fu2 = pm.FlatUpdate(case["offsets"], case["counts"], case["tau_fwd"], case["tau_bkwd"], optimizer=optimizer,
                            alpha=0.01 if optimizer == "sgdm" else 5e-4, K=32, D=0.5)
        t2 = {n: torch.from_numpy(case[n]).to(dev) for n in ("w", "m", "delta", "g")}
        t = t2                                                       # fresh state, so that the results still compare
        s = torch.from_numpy(case["s"]).to(dev) if optimizer == "adam" else None
        lp = torch.zeros(case["total"], dtype=torch.bfloat16, device=dev)
        call = fu2.pm_update_flat_static
        torch.cuda.synchronize()
        free0 = torch.cuda.mem_get_info(dev)[0]                      # the driver's own count of free device memory
        reserved0 = torch.cuda.memory_reserved(dev)
    for k in (9, 10):
        if stream is not None:
            stream.wait_stream(torch.cuda.current_stream(dev))
            call(t["w"], t["m"], s, t["delta"], t["g"], lp, k, stream=stream)
            stream.synchronize()
        else:
            call(t["w"], t["m"], s, t["delta"], t["g"], lp, k)
        if static and check_no_alloc:
            torch.cuda.synchronize()
            assert torch.cuda.mem_get_info(dev)[0] == free0 and torch.cuda.memory_reserved(dev) == reserved0
        torch.cuda.synchronize()
        snap = {n: t[n].cpu().numpy().copy() for n in ("w", "m", "delta")}
        if s is not None:
            snap["s"] = s.cpu().numpy().copy()
        snap["w_lp"] = lp.float().cpu().numpy().copy()
        snaps.append(snap)
    return snaps


@pytest.mark.parametrize("optimizer,n,P", [("sgdm", 200003, 8), ("adam", 70001, 64), ("sgdm", 300000, 256)])
def test_static_variant_matches_workspace_variant_on_two_calls(cuda_device, optimizer, n, P):
    case = I.update_sweep_case(n, P, optimizer)
    ref = run_two_calls(case, optimizer, static=False)
    got = run_two_calls(case, optimizer, static=True)
    for call in range(2):
        for name in ref[call]:
            np.testing.assert_array_equal(got[call][name].view(np.uint32), ref[call][name].view(np.uint32),
                                          err_msg=f"call {call} {name}")
    assert np.abs(ref[1]["w"] - ref[0]["w"]).max() > 0          # the second call did advance the state


def test_static_variant_after_a_different_stage_split(cuda_device):
    # a call with many stages leaves a long table behind; a following call with few stages must not see it
    big = I.update_sweep_case(100000, 200, "sgdm")
    run_two_calls(big, "sgdm", static=True)
    small = I.update_sweep_case(50000, 3, "sgdm")
    ref = run_two_calls(small, "sgdm", static=False)
    got = run_two_calls(small, "sgdm", static=True)
    for name in ref[1]:
        np.testing.assert_array_equal(got[1][name].view(np.uint32), ref[1][name].view(np.uint32), err_msg=name)


def test_static_variant_rejects_more_stages_than_it_holds(cuda_device):
    import torch
    import paper_1910_05124_b200 as pm
    assert pm.lib().pm_update_flat_static_max_stages() == 256
    case = I.update_sweep_case(100000, 257, "sgdm")
    dev = torch.device("cuda:0")
    t = {n: torch.from_numpy(case[n]).to(dev) for n in ("w", "m", "delta", "g")}
    fu = pm.FlatUpdate(case["offsets"], case["counts"], case["tau_fwd"], case["tau_bkwd"], optimizer="sgdm", alpha=0.01)
    before = t["w"].clone()
    with pytest.raises(pm.PipeMareError, match="at most 256 stages"):
        fu.pm_update_flat_static(t["w"], t["m"], None, t["delta"], t["g"], None, 0)
    torch.cuda.synchronize()
    assert torch.equal(before, t["w"])


def test_static_variant_allocates_nothing_and_takes_any_stream(cuda_device):
    """Adam at the 256-stage limit, on a stream of the caller's: the driver reports the same free device memory
    before and after each call (and torch's pool has not grown), and the bits equal the workspace variant's."""
    import torch
    case = I.update_sweep_case(260000, 256, "adam")
    ref = run_two_calls(case, "adam", static=False)
    side = torch.cuda.Stream()
    got = run_two_calls(case, "adam", static=True, stream=side, check_no_alloc=True)
    for call in range(2):
        for name in ref[call]:
            np.testing.assert_array_equal(got[call][name].view(np.uint32), ref[call][name].view(np.uint32),
                                          err_msg=f"call {call} {name}")
