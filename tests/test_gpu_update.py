"""GPU parity of the fused PipeMare update (pm_update_flat) against the oracle, bit for bit."""
import numpy as np
import pytest

import pm_inputs as I
from oracle import update as U
from oracle.bf16 import bf16_round

pytestmark = pytest.mark.gpu


def oracle_update(case, hp, k):
    out = {name: case[name].copy() for name in ("w", "m", "delta")}
    if hp["optimizer"] == "adam":
        out["s"] = case["s"].copy()
    for i, (o, c) in enumerate(zip(case["offsets"], case["counts"])):
        sl = slice(o, o + c)
        st = {"v": case["m"][sl]} if hp["optimizer"] == "sgdm" else {"m": case["m"][sl], "s": case["s"][sl]}
        w1, st1, d1 = U.pipemare_update(case["w"][sl], st, case["delta"][sl], case["g"][sl], k=k,
                                        tau_fwd=case["tau_fwd"][i], tau_bkwd=case["tau_bkwd"][i], hp=hp)
        out["w"][sl], out["delta"][sl] = w1, d1
        if hp["optimizer"] == "sgdm":
            out["m"][sl] = st1["v"]
        else:
            out["m"][sl], out["s"][sl] = st1["m"], st1["s"]
    return out


def gpu_update(case, hp, k, with_lp=True, calls=1):
    import torch
    import paper_1910_05124_b200 as pm
    dev = torch.device("cuda:0")
    t = {n: torch.from_numpy(case[n]).to(dev) for n in ("w", "m", "delta", "g")}
    s = torch.from_numpy(case["s"]).to(dev) if hp["optimizer"] == "adam" else None
    lp = torch.zeros(case["total"], dtype=torch.bfloat16, device=dev) if with_lp else None
    fu = pm.FlatUpdate(case["offsets"], case["counts"], case["tau_fwd"], case["tau_bkwd"], optimizer=hp["optimizer"],
                       alpha=hp["alpha"], beta1=hp["beta1"], beta2=hp["beta2"], eps=hp["eps"], t1=hp["t1"], K=hp["K"],
                       t2=hp["t2"], D=hp["D"])
    for c in range(calls):
        fu.pm_update_flat(t["w"], t["m"], s, t["delta"], t["g"], lp, k + c)
    torch.cuda.synchronize()
    out = {n: t[n].cpu().numpy() for n in ("w", "m", "delta")}
    if s is not None:
        out["s"] = s.cpu().numpy()
    if lp is not None:
        out["w_lp"] = lp.float().cpu().numpy()
    return out


def hp_(optimizer, **kw):
    hp = dict(optimizer=optimizer, alpha=0.01 if optimizer == "sgdm" else 5e-4, beta1=0.9, beta2=0.98, eps=1e-8,
              t1=True, K=32, t2=True, D=0.5)
    hp.update(kw)
    return hp


@pytest.mark.parametrize("optimizer", ["sgdm", "adam"])
@pytest.mark.parametrize("n,P", [(1000, 8), (100003, 8), (1 << 20, 64), (1000000, 512), (3000017, 64)])
def test_update_matches_oracle_bitwise(cuda_device, optimizer, n, P):
    case = I.update_sweep_case(n, P, optimizer)
    hp = hp_(optimizer)
    k = 16                                                  # 0 < p < 1: exercises tau^p
    ref = oracle_update(case, hp, k)
    got = gpu_update(case, hp, k)
    for name in ref:
        np.testing.assert_array_equal(got[name].view(np.uint32), ref[name].view(np.uint32), err_msg=name)
    np.testing.assert_array_equal(got["w_lp"], bf16_round(ref["w"]).astype(np.float32))


@pytest.mark.parametrize("optimizer", ["sgdm", "adam"])
@pytest.mark.parametrize("kw", [dict(t1=False), dict(t2=False), dict(t1=False, t2=False), dict(K=1), dict(D=0.1)])
def test_update_variants_match_oracle(cuda_device, optimizer, kw):
    case = I.update_sweep_case(50000, 8, optimizer)
    hp = hp_(optimizer, **kw)
    for k in (0, 5, 40):
        ref = oracle_update(case, hp, k)
        got = gpu_update(case, hp, k, with_lp=False)
        for name in ref:
            np.testing.assert_array_equal(got[name].view(np.uint32), ref[name].view(np.uint32), err_msg=f"{name} k={k}")


@pytest.mark.parametrize("k", [3, 2000])
def test_adam_on_zero_and_denormal_state_matches_oracle_bitwise(cuda_device, k):
    """Parameters that have seen no gradient yet (g = m = s = 0: untouched embedding rows), negative zeros, moments
    that have decayed into the denormal range and zero weights: the kernel keeps the zeros out of its division and
    square-root sequences, and the bits must still be those of the plain formula.  At k = 2000 both bias corrections
    have rounded to 1."""
    case = I.update_sweep_case(40000, 4, "adam")
    n = case["total"]
    idx = np.arange(n)
    valid = np.zeros(n, dtype=bool)                          # the padding behind each stage stays zero
    for o, c in zip(case["offsets"], case["counts"]):
        valid[o:o + c] = True
    zero = ((idx // 512) % 3 == 0) & valid                   # whole rows of zeros
    for name in ("g", "m", "s"):
        case[name][zero] = 0.0
    case["m"][(idx % 512 == 7) & zero] = -0.0
    case["g"][(idx % 512 == 9) & zero] = -0.0
    den = ((idx // 512) % 3 == 1) & valid
    tiny = np.float32(1e-45)
    case["m"][den & (idx % 4 == 0)] = tiny                   # smallest denormal, both signs
    case["m"][den & (idx % 4 == 1)] = -tiny
    case["s"][den & (idx % 4 < 2)] = tiny
    case["g"][den & (idx % 4 < 2)] = 0.0
    case["s"][den & (idx % 4 == 2)] = np.float32(3e-39)      # denormal second moment under a normal first moment
    case["w"][(idx % 64 == 5)] = 0.0                         # zero weights (biases) take the step as it is
    hp = hp_("adam")
    with np.errstate(all="ignore"):
        ref = oracle_update(case, hp, k)
    got = gpu_update(case, hp, k)
    for name in ref:
        np.testing.assert_array_equal(got[name].view(np.uint32), ref[name].view(np.uint32), err_msg=name)


def test_update_with_equal_delays_leaves_delta_alone(cuda_device):
    # tau_fwd = tau_bkwd (weight-stashing style delays): no gap, so no correction state is kept
    case = I.update_sweep_case(20000, 4, "sgdm")
    case["tau_bkwd"] = list(case["tau_fwd"])
    hp = hp_("sgdm")
    ref = oracle_update(case, hp, 3)
    got = gpu_update(case, hp, 3)
    np.testing.assert_array_equal(got["delta"], case["delta"])
    np.testing.assert_array_equal(got["w"].view(np.uint32), ref["w"].view(np.uint32))


def test_two_calls_in_a_row_advance_state(cuda_device):
    case = I.update_sweep_case(70000, 8, "adam")
    hp = hp_("adam")
    ref = oracle_update(case, hp, 7)
    case2 = dict(case)
    case2.update(w=ref["w"], m=ref["m"], s=ref["s"], delta=ref["delta"])
    ref2 = oracle_update(case2, hp, 8)
    got = gpu_update(case, hp, 7, calls=2)
    for name in ref2:
        np.testing.assert_array_equal(got[name].view(np.uint32), ref2[name].view(np.uint32), err_msg=name)


def test_padding_stays_zero_and_gradients_untouched(cuda_device):
    case = I.update_sweep_case(1000, 8, "adam")
    got = gpu_update(case, hp_("adam"), 2)
    for i, (o, c) in enumerate(zip(case["offsets"], case["counts"])):
        end = case["offsets"][i + 1] if i + 1 < len(case["offsets"]) else case["total"]
        assert (got["w"][o + c:end] == 0).all() and (got["m"][o + c:end] == 0).all()


def test_flat_update_rejects_bad_arguments(cuda_device):
    import torch
    import paper_1910_05124_b200 as pm
    case = I.update_sweep_case(1000, 4, "sgdm")
    dev = torch.device("cuda:0")
    t = {n: torch.from_numpy(case[n]).to(dev) for n in ("w", "m", "delta", "g")}
    fu = pm.FlatUpdate([0, 100, 512, 768], case["counts"], case["tau_fwd"], case["tau_bkwd"], optimizer="sgdm", alpha=0.01)
    with pytest.raises(pm.PipeMareError, match="multiples of 64"):
        fu.pm_update_flat(t["w"], t["m"], None, t["delta"], t["g"], None, 0)
    fu = pm.FlatUpdate(case["offsets"], case["counts"], case["tau_fwd"], case["tau_bkwd"], optimizer="adam", alpha=0.01)
    with pytest.raises(pm.PipeMareError, match="missing arena"):
        fu.pm_update_flat(t["w"], t["m"], None, t["delta"], t["g"], None, 0)
