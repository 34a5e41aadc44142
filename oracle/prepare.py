"""Oracle of the token preparation that feeds the fast-weight update (TEST INFRASTRUCTURE ONLY).

What the model does upstream of the chunk update (Section 4, "Overall Architecture" and the gate parameterisation):
queries and keys pass through SiLU and are then L2-normalised per token and head; the gates come from logits
(outputs of small linear heads) as

    eta_t   = eta_base * sigmoid(a_t)                         (Eq. "eta_parameterization")
    beta_t  = sigmoid(b_t) ** (1 / tau)                       (Eq. "beta_parameterization")
    alpha_t = alpha_base * sigmoid(c_t),  gamma_t = 1 - eta_t * alpha_t      (Eq. "decay_derivation")

Reading: the paper does not say how a zero vector is normalised; x / max(||x||_2, eps) is taken (what the common
library routine does), eps an argument.  Plain numpy, fp64.  The reverse pass is written out by hand; the tests pin
both directions against torch's own ops and autograd.
"""
from __future__ import annotations

import numpy as np


def _sigmoid(z):
    return 1.0 / (1.0 + np.exp(-z))


def silu_l2norm(x, eps=1e-12):
    """x [..., d] -> silu(x) / max(||silu(x)||, eps) along the last axis."""
    x = np.asarray(x, dtype=np.float64)
    s = x * _sigmoid(x)
    n = np.sqrt((s * s).sum(-1, keepdims=True))
    return s / np.maximum(n, eps)


def silu_l2norm_vjp(x, y_bar, eps=1e-12):
    """Adjoint of silu_l2norm: y = s / m, m = max(||s||, eps); for ||s|| > eps  s_bar = (y_bar - y <y_bar, y>) / m."""
    x = np.asarray(x, dtype=np.float64)
    y_bar = np.asarray(y_bar, dtype=np.float64)
    sg = _sigmoid(x)
    s = x * sg
    n = np.sqrt((s * s).sum(-1, keepdims=True))
    m = np.maximum(n, eps)
    y = s / m
    proj = (y_bar * y).sum(-1, keepdims=True)
    s_bar = np.where(n > eps, (y_bar - y * proj) / m, y_bar / m)
    return s_bar * (sg * (1.0 + x * (1.0 - sg)))          # silu'(x) = sigma (1 + x (1 - sigma))


def gates(a, b, c, eta_base, tau, alpha_base):
    """Logits -> (eta, beta, gamma)."""
    a, b, c = (np.asarray(t, dtype=np.float64) for t in (a, b, c))
    eta = eta_base * _sigmoid(a)
    beta = _sigmoid(b) ** (1.0 / tau)
    alpha = alpha_base * _sigmoid(c)
    return eta, beta, 1.0 - eta * alpha


def gates_vjp(a, b, c, eta_base, tau, alpha_base, d_eta, d_beta, d_gamma):
    """Adjoints of the three logits."""
    a, b, c, d_eta, d_beta, d_gamma = (np.asarray(t, dtype=np.float64) for t in (a, b, c, d_eta, d_beta, d_gamma))
    sa, sb, sc = _sigmoid(a), _sigmoid(b), _sigmoid(c)
    eta = eta_base * sa
    beta = sb ** (1.0 / tau)
    alpha = alpha_base * sc
    eta_bar = d_eta - d_gamma * alpha                      # gamma = 1 - eta alpha
    alpha_bar = -d_gamma * eta
    da = eta_bar * eta_base * sa * (1.0 - sa)
    db = d_beta * beta * (1.0 - sb) / tau                  # d/db sigma^(1/tau) = (1/tau) sigma^(1/tau) (1 - sigma)
    dc = alpha_bar * alpha_base * sc * (1.0 - sc)
    return da, db, dc
