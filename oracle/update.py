"""The per-stage PipeMare weight update, element-wise, in a chosen precision.

TEST INFRASTRUCTURE (see package docstring).

Follows, in this order:
  * T1 (Section 3.1, Eq. 2):  alpha_{k,i} = alpha_{k,base} / tau_i^{p_k},  p_k = 1 - min(k/K, 1)
  * momentum SGD (Appendix B.3):  v <- beta v - alpha g ;  w' = w + v
    or bias-corrected Adam (Table 8 names the optimiser and its betas)
  * T2 accumulator (Section 3.2):  delta <- gamma delta + (1-gamma)(w' - w),
    gamma_i = D^{1/(tau_fwd,i - tau_bkwd,i)}
  * T2 corrected backward weights:  u_bkwd = w - (tau_fwd - tau_bkwd) delta

Precision: state arrays have dtype `dt` (float32 for the configured
workloads, whose state precision the workload fixes; float64 in the
closed-form pins).  Per-stage scalars are computed in float64 and then cast
to `dt`.  Every array operation below is a single numpy ufunc, so each is
rounded once in `dt`, in the order written, with no fused multiply-add.

Readings where the paper is silent:
  * tau = 0: the step size is not rescaled (max(tau,1)), gamma := 0 is never
    used because the correction and the accumulator refresh are skipped.
  * k counts updates from 0, so p_0 = 1 and p_k = 0 for k >= K.
  * Adam: bias-corrected, no weight decay; m_hat = m/(1-beta1^(k+1)),
    s_hat = s/(1-beta2^(k+1)), w' = w - (alpha m_hat)/(sqrt(s_hat)+eps).

Pins: tests/test_oracle_update.py (T1 table values, gamma table values,
scalar closed forms through the recurrence, hand-computed single steps).
"""
import numpy as np


def t1_exponent(k, K):
    """p_k = 1 - min(k/K, 1)   (Eq. 2)."""
    return 1.0 - min(k / K, 1.0)


def t1_step_size(alpha_base, tau_fwd, k, K, enabled=True):
    """alpha_{k,i} = alpha_{k,base} / tau_i^{p_k}   (Eq. 2); float64."""
    if not enabled:
        return float(alpha_base)
    return float(alpha_base) / float(max(tau_fwd, 1)) ** t1_exponent(k, K)


def t2_gamma(D, tau_fwd, tau_bkwd):
    """gamma_i = D^{1/(tau_fwd,i - tau_bkwd,i)}   (T2); float64.  Undefined (returns None) at zero gap."""
    gap = tau_fwd - tau_bkwd
    if gap == 0:
        return None
    return float(D) ** (1.0 / gap)


def corrected_backward_weights(w_bkwd, delta, tau_fwd, tau_bkwd, enabled=True):
    """u_bkwd = w_{t - tau_bkwd} - (tau_fwd - tau_bkwd) * delta_t   (T2)."""
    gap = tau_fwd - tau_bkwd
    if not enabled or gap == 0:
        return w_bkwd
    dt = w_bkwd.dtype.type
    return w_bkwd - dt(gap) * delta


def sgdm_step(w, v, g, alpha, beta):
    """v' = beta v - alpha g ;  w' = w + v'   (Appendix B.3).  Returns (w', v')."""
    dt = w.dtype.type
    v_new = dt(beta) * v - dt(alpha) * g
    return w + v_new, v_new


def adam_step(w, m, s, g, alpha, beta1, beta2, eps, k):
    """Bias-corrected Adam at update index k (0-based).  Returns (w', m', s')."""
    dt = w.dtype.type
    b1, b2 = dt(beta1), dt(beta2)
    m_new = b1 * m + (dt(1) - b1) * g
    s_new = b2 * s + (dt(1) - b2) * (g * g)
    bc1 = dt(1.0 - float(b1) ** (k + 1))
    bc2 = dt(1.0 - float(b2) ** (k + 1))
    m_hat = m_new / bc1
    s_hat = s_new / bc2
    w_new = w - (dt(alpha) * m_hat) / (np.sqrt(s_hat) + dt(eps))
    return w_new, m_new, s_new


def delta_refresh(delta, w_new, w_old, gamma):
    """delta' = gamma delta + (1 - gamma)(w' - w)   (T2)."""
    dt = delta.dtype.type
    g = dt(gamma)
    return g * delta + (dt(1) - g) * (w_new - w_old)


def pipemare_update(w, opt_state, delta, g, *, k, tau_fwd, tau_bkwd, hp, k_t1=None):
    """One update of one tensor of one stage.  Returns (w', opt_state', delta').

    hp: dict with optimizer ('sgdm'|'adam'), alpha (float or callable k -> float),
    beta1, beta2, eps, t1 (bool), K, t2 (bool), D.
    k indexes the base step size and Adam's bias correction; k_t1 (default k) is the step the T1 annealing counts
    from (after synchronous warm-up epochs, Section 4, the annealing starts where PipeMare starts).
    """
    alpha_base = hp["alpha"](k) if callable(hp["alpha"]) else hp["alpha"]
    alpha = t1_step_size(alpha_base, tau_fwd, k if k_t1 is None else k_t1, hp["K"], hp["t1"])
    if hp["optimizer"] == "sgdm":
        w_new, v_new = sgdm_step(w, opt_state["v"], g, alpha, hp["beta1"])
        new_state = {"v": v_new}
    elif hp["optimizer"] == "adam":
        w_new, m_new, s_new = adam_step(w, opt_state["m"], opt_state["s"], g, alpha,
                                        hp["beta1"], hp["beta2"], hp["eps"], k)
        new_state = {"m": m_new, "s": s_new}
    else:
        raise ValueError(hp["optimizer"])
    gamma = t2_gamma(hp["D"], tau_fwd, tau_bkwd) if hp["t2"] else None
    delta_new = delta if gamma is None else delta_refresh(delta, w_new, w, gamma)
    return w_new, new_state, delta_new


def fresh_opt_state(w, optimizer):
    z = np.zeros_like(w)
    return {"v": z} if optimizer == "sgdm" else {"m": z, "s": z.copy()}
