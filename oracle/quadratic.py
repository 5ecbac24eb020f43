"""Gradient samples of the one-dimensional quadratic models (Sections 3, 3.1, 3.2).

TEST INFRASTRUCTURE (see package docstring).

    f(w) = lambda w^2 / 2
    no discrepancy:   grad = lambda * u_fwd - eta_t                      (Section 3)
    with discrepancy: grad = (lambda + Delta) u_fwd - Delta u_bkwd - eta_t   (Section 3.2)
    with recomputation: grad = (lambda + Delta) u_fwd - (Delta - Phi) u_bkwd - Phi u_recomp - eta_t   (Appendix D)

These plug into recurrence.run as a single stage holding one scalar, so the
stability lemmas and characteristic polynomials of the paper test the very
loop the network workloads go through.
"""
import numpy as np


def quadratic_grad(lam, Delta=0.0, noise=None, Phi=0.0):
    """Return grad_fn for recurrence.run; noise: optional callable t -> eta_t.  Phi: sensitivity to the weights the
    recomputation used (needs recurrence.run(..., tau_recomp=...) when non-zero)."""
    def grad_fn(t, u_fwd, u_bkwd, u_recomp=None):
        wf = u_fwd[0][0]
        wb = u_bkwd[0][0]
        eta = 0.0 if noise is None else noise(t)
        g = (lam + Delta) * wf - (Delta - Phi) * wb - eta
        if Phi != 0.0:
            g = g - Phi * u_recomp[0][0]
        return float(0.5 * lam * wf[0] ** 2), [[np.asarray(g)]]
    return grad_fn
