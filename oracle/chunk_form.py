"""Matrix form of one chunk update for the GELU-MLP fast weights (numpy), with optional rounding hooks.

TEST INFRASTRUCTURE ONLY, like the rest of oracle/.  The sequential oracle (e2ttt_oracle.c) runs the token-wise
recurrence literally; this module evaluates the same chunk the way Algorithm 1 states it: one inner forward and
backward for all tokens of the chunk at the chunk-start weights (Section 3.1, Appendix "Single Backward Pass for
Both Aggregates"), the scalar kernels K^W, K^M and the three carries (Eq. "scalar_aux", evaluated by the division-free
recurrence S_t = beta_{t+1} S_{t+1} + gt_t with S_t = bt_t R_t, the inner sum of Eq. "unroll_recurrence"), and the
closed-form transition of Proposition 1.  It serves three purposes:

  * with dtype = float64 and no hooks it must reproduce the sequential oracle (a pin of both);
  * with dtype = float32 it is the closed form "in fp32", compared with sequential_from_grads() in fp32 over many
    chunks: the numerical-equivalence experiment of Section 3.2 / Appendix "Exactness" on synthetic inputs;
  * with hooks it rounds, in otherwise fp64 arithmetic, exactly where a bf16 tensor-core implementation of the chunk
    declares that it rounds (operand copies of W, the activation tile, pu, the scaled operands of the aggregations,
    the output).  A GPU result then differs from the hooked value only by accumulation order and the fp32 state:
    a sharp test for indexing and synchronisation mistakes, next to the unhooked comparison, which is the accuracy
    statement.

Nothing here is shared with the CUDA path.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
from scipy.special import erf


def round_bf16(x):
    """Nearest bf16 (ties to even) of fp32-representable values, returned in the input's dtype."""
    a = np.ascontiguousarray(x, dtype=np.float32)
    u = a.view(np.uint32)
    r = ((u + (((u >> 16) & 1) + np.uint32(0x7FFF))) & np.uint32(0xFFFF0000)).astype(np.uint32)
    return r.view(np.float32).astype(np.asarray(x).dtype if np.asarray(x).dtype.kind == "f" else np.float64)


def round_f16(x):
    return np.asarray(x, dtype=np.float64).astype(np.float16).astype(np.asarray(x).dtype)


@dataclass
class Hooks:
    """Where a bf16 tensor-core implementation rounds.  `gelu` selects the activation formula it evaluates: "erf" is the
    exact form of the paper's reading, "tanh" the usual tanh approximation (an implementation that uses it declares it)."""
    operands: bool = True       # W1, W2 as bf16 operand copies (the state itself stays unrounded)
    activations: bool = True    # gelu(Z) -> bf16 before the second product
    pu: bool = True             # dL/du -> bf16 before the backward product and the W2 aggregation
    scaled: bool = True         # kW a, kM a (from an fp16 copy of a), kW pz, kM pz -> bf16 before the aggregations
    output: bool = True         # o -> bf16
    gelu: str = "tanh"


def _id(x):
    return x


def gelu_pair(z, form):
    """gelu(z) and gelu'(z) in the dtype of z."""
    dt = z.dtype
    if form == "erf":
        zz = z.astype(np.float64)
        Phi = 0.5 * (1.0 + erf(zz / np.sqrt(2.0)))
        phi = np.exp(-0.5 * zz * zz) / np.sqrt(2.0 * np.pi)
        return (zz * Phi).astype(dt), (Phi + zz * phi).astype(dt)
    c0, c1 = dt.type(0.7978845608028654), dt.type(0.044715)
    u = c0 * (z + c1 * z * z * z)
    t = np.tanh(u)
    du = c0 * (dt.type(1.0) + dt.type(3.0) * c1 * z * z)
    half = dt.type(0.5)
    return half * z * (dt.type(1.0) + t), half * (dt.type(1.0) + t) + half * z * (dt.type(1.0) - t * t) * du


def scalar_kernels(eta, beta, gamma, dtype=np.float64):
    """K^W_t, K^M_t (t = 1..C) and the carries cw = gt_0, cm = bt_0 R_1, cb = bt_0 by the division-free suffix recurrence."""
    eta, beta, gamma = (np.asarray(a, dtype=dtype) for a in (eta, beta, gamma))
    C = eta.shape[0]
    one = dtype(1.0)
    bt = np.empty(C + 1, dtype); gt = np.empty(C + 1, dtype); S = np.empty(C + 1, dtype)
    bt[C] = gt[C] = S[C] = one
    for t in range(C - 1, -1, -1):          # index t = the paper's t; beta[t] is the paper's beta_{t+1}
        gt[t] = gamma[t] * gt[t + 1]
        bt[t] = beta[t] * bt[t + 1]
        S[t] = beta[t] * S[t + 1] + gt[t]
    return eta * S[1:], eta * bt[1:], gt[0], beta[0] * S[1], bt[0]


def layer_norm_rows(U, eps):
    dt = U.dtype
    mu = U.mean(axis=1, keepdims=True, dtype=dt)
    c = U - mu
    var = (c * c).mean(axis=1, keepdims=True, dtype=dt)
    r = dt.type(1.0) / np.sqrt(var + dt.type(eps))
    return c * r, r


def chunk_mlp(K, Q, V, eta, beta, gamma, W1, W2, M1, M2, eps=1e-5, dtype=np.float64, hooks: Hooks | None = None):
    """One chunk (rows = tokens).  Returns o, (W1', W2', M1', M2') and the per-token pieces (Pu, A, Pz) of the gradients.

    Per-token negative gradients are G_t(W2) = -pu_t (x) a_t and G_t(W1) = -pz_t (x) k_t; the transition is Proposition 1.
    """
    dt = np.dtype(dtype)
    K, Q, V, W1, W2, M1, M2 = (np.asarray(a, dtype=dt) for a in (K, Q, V, W1, W2, M1, M2))
    form = hooks.gelu if hooks else "erf"
    r16 = (lambda x: round_bf16(x).astype(dt)) if hooks else _id
    W1o = r16(W1) if hooks and hooks.operands else W1
    W2o = r16(W2) if hooks and hooks.operands else W2
    kW, kM, cw, cm, cb = scalar_kernels(eta, beta, gamma, dt.type)

    def net_u(X):
        Z = X @ W1o.T
        a, da = gelu_pair(Z, form)
        A = r16(a) if hooks and hooks.activations else a
        return Z, a, da, A, A @ W2o.T

    # outputs from the chunk-start weights (Algorithm 1 line 1)
    _, _, _, _, Uq = net_u(Q)
    Yq, _ = layer_norm_rows(Uq, eps)
    o = Q + Yq
    if hooks and hooks.output:
        o = r16(o)
    # inner forward and backward at the chunk-start weights, all tokens at once
    _, a, da, A, Uk = net_u(K)
    Yk, r = layer_norm_rows(Uk, eps)
    E = K + Yk - V                                        # dL_t/dy for L_t = 1/2 ||f(k_t) - v_t||^2
    Pu = r * (E - E.mean(axis=1, keepdims=True, dtype=dt) - Yk * (E * Yk).mean(axis=1, keepdims=True, dtype=dt))
    if hooks and hooks.pu:
        Pu = r16(Pu)
    Pz = (Pu @ W2o) * da
    if hooks and hooks.scaled:
        a16 = round_f16(a).astype(dt)
        AkW, AkM = r16(kW[:, None] * a16), r16(kM[:, None] * a16)
        PzW, PzM = r16(kW[:, None] * Pz), r16(kM[:, None] * Pz)
    else:
        src = A if hooks else a
        AkW, AkM = kW[:, None] * src, kM[:, None] * src
        PzW, PzM = kW[:, None] * Pz, kM[:, None] * Pz
    # Proposition 1: W_C = cw W_0 + cm M_0 + sum_t K^W_t G_t,  M_C = cb M_0 + sum_t K^M_t G_t
    W2n = cw * W2 + cm * M2 - Pu.T @ AkW
    M2n = cb * M2 - Pu.T @ AkM
    W1n = cw * W1 + cm * M1 - PzW.T @ K
    M1n = cb * M1 - PzM.T @ K
    return o, (W1n, W2n, M1n, M2n), dict(Pu=Pu, A=a, Pz=Pz, kW=kW, kM=kM)


def forward_mlp(q, k, v, eta, beta, gamma, W1, W2, M1, M2, C, eps=1e-5, dtype=np.float64, hooks: Hooks | None = None):
    """All chunks of ONE sequence (arrays [L, d], [L]); the state is carried in `dtype` (fp32 master when hooked:
    pass dtype=np.float64 with hooks for "fp64 arithmetic, rounding only at the hooks")."""
    L = q.shape[0]
    outs = []
    st = tuple(np.asarray(a, dtype=dtype) for a in (W1, W2, M1, M2))
    for s in range(0, L, C):
        e = min(L, s + C)
        o, st, _ = chunk_mlp(k[s:e], q[s:e], v[s:e], eta[s:e], beta[s:e], gamma[s:e], st[0], st[1], st[2], st[3], eps, dtype, hooks)
        outs.append(o)
    return np.concatenate(outs, axis=0), st


def sequential_from_grads(W0, M0, G, eta, beta, gamma, dtype=np.float64):
    """Eq. "tokenwise_ttt_decay_momentum" run literally in `dtype` over the per-token gradients G[t] of ONE matrix:
    M_t = beta_t M_{t-1} + eta_t G_t,  W_t = gamma_t W_{t-1} + M_t."""
    W = np.asarray(W0, dtype=dtype).copy()
    M = np.asarray(M0, dtype=dtype).copy()
    for t in range(len(G)):
        M = dtype(beta[t]) * M + dtype(eta[t]) * np.asarray(G[t], dtype=dtype)
        W = dtype(gamma[t]) * W + M
    return W, M
