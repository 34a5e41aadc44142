"""Direct fp64 evaluations of the paper's closed forms for ONE chunk (numpy, O(C^2) and proud of it).

TEST INFRASTRUCTURE ONLY, like the rest of oracle/.  Two independent statements of the chunk-end
states, both written straight from the paper, used to cross-check the sequential oracle:

  * proposition()  - Proposition 1 (Eq. "Mc_closed", "Wc_closed") with the suffix products and the
    ratio sum of Eq. "scalar_aux", exactly as printed (it divides by the beta suffix product, so it
    needs beta > 0 and a product that does not underflow);
  * unrolled()     - Eq. "unroll_recurrence": explicit products, no division, valid for beta = 0.

Neither calls the sequential oracle; they only combine per-token gradients G_t handed in by the caller.
"""
from __future__ import annotations

import numpy as np


def scalar_aux(beta, gamma):
    """Eq. "scalar_aux": bt_t = prod_{i>t} beta_i, gt_t likewise, R_t = sum_{i=t..C} gt_i / bt_i, t = 0..C.

    Index t of the returned arrays is the paper's t (0..C); beta[0] is the paper's beta_1.
    R_0 is returned for completeness but the paper never uses it.
    """
    beta = np.asarray(beta, dtype=np.float64)
    gamma = np.asarray(gamma, dtype=np.float64)
    C = beta.shape[0]
    bt = np.ones(C + 1)
    gt = np.ones(C + 1)
    for t in range(C + 1):
        for i in range(t + 1, C + 1):
            bt[t] *= beta[i - 1]
            gt[t] *= gamma[i - 1]
    R = np.zeros(C + 1)
    for t in range(C + 1):
        for i in range(max(t, 0), C + 1):
            R[t] += gt[i] / bt[i]
    return bt, gt, R


def kernels(eta, beta, gamma):
    """K^M_t = eta_t bt_t, K^W_t = eta_t bt_t R_t (t = 1..C) and the three carries of Algorithm 1 lines 6-7."""
    eta = np.asarray(eta, dtype=np.float64)
    bt, gt, R = scalar_aux(beta, gamma)
    KM = eta * bt[1:]
    KW = eta * bt[1:] * R[1:]
    return KW, KM, dict(cw=gt[0], cm=bt[0] * R[1], cb=bt[0])


def proposition(W0, M0, G, eta, beta, gamma):
    """Proposition 1.  W0, M0: lists of matrices; G: list over tokens of lists of matrices."""
    KW, KM, c = kernels(eta, beta, gamma)
    WC = [c["cw"] * w + c["cm"] * m for w, m in zip(W0, M0)]
    MC = [c["cb"] * m for m in M0]
    for t, Gt in enumerate(G):
        for i, g in enumerate(Gt):
            WC[i] = WC[i] + KW[t] * g
            MC[i] = MC[i] + KM[t] * g
    return WC, MC


def unrolled(W0, M0, G, eta, beta, gamma):
    """Eq. "unroll_recurrence" for W_C and the t = C case of the unrolled momentum, products written out."""
    eta = np.asarray(eta, dtype=np.float64)
    beta = np.asarray(beta, dtype=np.float64)
    gamma = np.asarray(gamma, dtype=np.float64)
    C = eta.shape[0]

    def prod(x, lo, hi):  # prod_{i=lo..hi} x_i, 1-based, empty = 1
        p = 1.0
        for i in range(lo, hi + 1):
            p *= x[i - 1]
        return p

    decay = prod(gamma, 1, C)
    mom = sum(prod(beta, 1, t) * prod(gamma, t + 1, C) for t in range(1, C + 1))
    WC = [decay * w + mom * m for w, m in zip(W0, M0)]
    MC = [prod(beta, 1, C) * m for m in M0]
    for t in range(1, C + 1):
        wgt = sum(prod(beta, t + 1, j) * prod(gamma, j + 1, C) for j in range(t, C + 1))
        for i, g in enumerate(G[t - 1]):
            WC[i] = WC[i] + eta[t - 1] * wgt * g
            MC[i] = MC[i] + eta[t - 1] * prod(beta, t + 1, C) * g
    return WC, MC
