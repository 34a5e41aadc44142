"""Pins for the fp64 oracle: every check compares it with something that is NOT the oracle.

 - finite differences of the inner loss (definition of G_t, Section 2 "Expressive Token-wise Update");
 - torch's own layer_norm / gelu / silu for the fast-weight networks (Section 4 "Fast-weight Network");
 - Proposition 1 and Eq. "unroll_recurrence" evaluated directly (oracle/closed_form.py);
 - the limits the paper states: beta, gamma -> 1 (Appendix "Stability of the Cumulative Kernel"),
   C -> 1 (token-wise update), neutral momentum/decay (plain chunk-wise step, Eq. "chunk_gradient");
 - the hand-expanded C = 2 case (tests/golden/c2_coefficients.txt);
 - an independent automatic-differentiation run of the sequential program (forward values and all
   ten gradient groups), plus finite differences of the oracle's own forward.
"""
import os

import numpy as np
import pytest
import torch

from oracle import closed_form, oracle
from paper_2608_21308_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
KINDS = [oracle.KIND_MLP, oracle.KIND_SWIGLU]


def tiny(kind, d=4, h=8, L=8, C=4, seed=1, m_std=0.05, w_std=0.5, N=1, **kw):
    r = inputs.Recipe(B=N, H=1, L=L, d=d, h=h, C=C, kind=kind, seed=seed, m_std=m_std, w_std=w_std, **kw)
    return r, inputs.generate(r, with_d_o=True, with_dstate=True)


def rel(a, b):
    return float(np.max(np.abs(np.asarray(a) - np.asarray(b))) / (np.max(np.abs(b)) + 1e-300))


# ---------------------------------------------------------------- P1: inner gradients vs finite differences
@pytest.mark.parametrize("kind", KINDS)
def test_inner_gradient_matches_central_differences(kind):
    r, x = tiny(kind, d=4, h=8)
    W = [w[0].astype(np.float64) for w in x["W"]]
    k, v = x["k"][0, 0].astype(np.float64), x["v"][0, 0].astype(np.float64)
    _, G = oracle.inner(W, k, v, kind)
    step = 1e-6
    for i, w in enumerate(W):
        fd = np.zeros_like(w)
        for idx in np.ndindex(w.shape):
            Wp = [a.copy() for a in W]
            Wm = [a.copy() for a in W]
            Wp[i][idx] += step
            Wm[i][idx] -= step
            fd[idx] = (oracle.inner(Wp, k, v, kind, want_grad=False)[0]
                       - oracle.inner(Wm, k, v, kind, want_grad=False)[0]) / (2 * step)
        assert rel(G[i], -fd) < 1e-7, f"matrix {i}"
        assert np.max(np.abs(fd)) > 1e-3  # the check is not vacuous


@pytest.mark.parametrize("kind", KINDS)
def test_inner_loss_is_half_squared_error_of_the_network(kind):
    r, x = tiny(kind)
    W = [w[0].astype(np.float64) for w in x["W"]]
    k, v = x["k"][0, 1].astype(np.float64), x["v"][0, 1].astype(np.float64)
    loss, _ = oracle.inner(W, k, v, kind, want_grad=False)
    f = oracle.net(W, k, kind)
    assert abs(loss - 0.5 * np.sum((f - v) ** 2)) < 1e-14


# ---------------------------------------------------------------- network forward vs library routines
@pytest.mark.parametrize("kind", KINDS)
def test_network_matches_torch_library_ops(kind):
    r, x = tiny(kind, d=8, h=16, w_std=0.7)
    W = [torch.tensor(w[0], dtype=torch.float64) for w in x["W"]]
    q = torch.tensor(x["q"][0, 3], dtype=torch.float64)
    F = torch.nn.functional
    if kind == oracle.KIND_MLP:
        u = W[1] @ F.gelu(W[0] @ q)  # exact (erf) GELU
    else:
        u = W[2] @ (F.silu(W[0] @ q) * (W[1] @ q))
    ref = q + F.layer_norm(u, (u.shape[0],), eps=1e-5)
    got = oracle.net([w.numpy() for w in W], q.numpy(), kind, eps=1e-5)
    assert rel(got, ref.numpy()) < 1e-13


def test_layernorm_eps_is_inside_the_square_root():
    # constant pre-activation => variance 0 => LN output 0 for any eps > 0, f(x) = x
    d, h = 4, 8
    W = [np.zeros((h, d)), np.zeros((d, h))]
    x = np.arange(1.0, 5.0)
    assert np.array_equal(oracle.net(W, x, oracle.KIND_MLP, eps=1e-5), x)


# ---------------------------------------------------------------- P2: sequential vs Proposition 1 vs unrolled form
def per_token_G(x, W0, kind, C, start=0):
    return [oracle.inner(W0, x["k"][0, start + t].astype(np.float64), x["v"][0, start + t].astype(np.float64), kind)[1]
            for t in range(C)]


@pytest.mark.parametrize("kind", KINDS)
@pytest.mark.parametrize("C", [1, 2, 7, 16])
def test_sequential_chunk_end_equals_closed_forms(kind, C):
    r, x = tiny(kind, d=4, h=8, L=C, C=C, seed=3)
    W0 = [w[0].astype(np.float64) for w in x["W"]]
    M0 = [m[0].astype(np.float64) for m in x["M"]]
    out = oracle.forward(x["q"], x["k"], x["v"], x["eta"], x["beta"], x["gamma"], x["W"], x["M"], C, kind)
    G = per_token_G(x, W0, kind, C)
    eta, beta, gamma = (x[n][0].astype(np.float64) for n in ("eta", "beta", "gamma"))
    for name, fn in (("proposition", closed_form.proposition), ("unrolled", closed_form.unrolled)):
        WC, MC = fn(W0, M0, G, eta, beta, gamma)
        for i in range(len(W0)):
            assert rel(out["W"][i][0], WC[i]) < 1e-10, (name, "W", i)
            assert rel(out["M"][i][0], MC[i]) < 1e-10, (name, "M", i)


# ---------------------------------------------------------------- P3 / P4: scalar kernels in the limits the paper states
def test_unit_gates_give_linear_ratio_sum():
    C = 12
    eta = np.linspace(0.01, 0.1, C)
    KW, KM, c = closed_form.kernels(eta, np.ones(C), np.ones(C))
    t = np.arange(1, C + 1)
    assert np.allclose(KW, eta * (C - t + 1), rtol=0, atol=1e-15)   # R_t -> C - t + 1
    assert np.allclose(KM, eta, rtol=0, atol=1e-15)
    assert (c["cw"], c["cb"], c["cm"]) == (1.0, 1.0, float(C))
    # bound of the appendix: K^W_t <= eta_base * C = 5.12 for eta_base = 1e-2, C = 512
    KW512, KM512, _ = closed_form.kernels(np.full(512, 1e-2), np.full(512, 0.999), np.full(512, 0.9999))
    assert KW512.max() <= 5.12 and KM512.max() <= 1e-2


def test_constant_gates_give_geometric_kernel():
    C, b, g, e = 9, 0.8, 0.95, 0.05
    KW, KM, c = closed_form.kernels(np.full(C, e), np.full(C, b), np.full(C, g))
    n = C - np.arange(1, C + 1) + 1
    assert np.allclose(KW, e * (g ** n - b ** n) / (g - b), rtol=1e-13)
    assert np.allclose(KM, e * b ** (n - 1), rtol=1e-13)
    assert np.isclose(c["cm"], b * (g ** C - b ** C) / (g - b), rtol=1e-13)


@pytest.mark.parametrize("kind", KINDS)
def test_unit_gates_sequential_state(kind):
    C = 6
    r, x = tiny(kind, L=C, C=C, seed=5)
    x["beta"][:] = 1.0
    x["gamma"][:] = 1.0
    W0 = [w[0].astype(np.float64) for w in x["W"]]
    M0 = [m[0].astype(np.float64) for m in x["M"]]
    G = per_token_G(x, W0, kind, C)
    out = oracle.forward(x["q"], x["k"], x["v"], x["eta"], x["beta"], x["gamma"], x["W"], x["M"], C, kind)
    for i in range(len(W0)):
        W_exp = W0[i] + C * M0[i] + sum(float(x["eta"][0, t]) * (C - t) * G[t][i] for t in range(C))
        M_exp = M0[i] + sum(float(x["eta"][0, t]) * G[t][i] for t in range(C))
        assert rel(out["W"][i][0], W_exp) < 1e-12
        assert rel(out["M"][i][0], M_exp) < 1e-12


# ---------------------------------------------------------------- P5: C = 1 is the token-wise update
@pytest.mark.parametrize("kind", KINDS)
def test_chunk_size_one_is_tokenwise_ttt(kind):
    L = 6
    r, x = tiny(kind, L=L, C=1, seed=7)
    out = oracle.forward(x["q"], x["k"], x["v"], x["eta"], x["beta"], x["gamma"], x["W"], x["M"], 1, kind)
    W = [w[0].astype(np.float64) for w in x["W"]]
    M = [m[0].astype(np.float64) for m in x["M"]]
    for t in range(L):
        # outputs read the weights BEFORE token t's update (chunk-start weights of a one-token chunk)
        o_t = oracle.net(W, x["q"][0, t].astype(np.float64), kind)
        assert rel(out["o"][0, t], o_t) < 1e-13
        _, G = oracle.inner(W, x["k"][0, t].astype(np.float64), x["v"][0, t].astype(np.float64), kind)
        e, b, g = (float(x[n][0, t]) for n in ("eta", "beta", "gamma"))
        M = [b * m + e * gi for m, gi in zip(M, G)]
        W = [g * w + m for w, m in zip(W, M)]
    for i in range(len(W)):
        assert rel(out["W"][i][0], W[i]) < 1e-12
        assert rel(out["M"][i][0], M[i]) < 1e-12


# ---------------------------------------------------------------- P6: neutral momentum and decay = plain chunk-wise step
@pytest.mark.parametrize("kind", KINDS)
def test_neutral_gates_reduce_to_plain_chunkwise_ttt(kind):
    C = 8
    r, x = tiny(kind, L=2 * C, C=C, seed=9)
    x["beta"][:] = 0.0
    x["gamma"][:] = 1.0
    out = oracle.forward(x["q"], x["k"], x["v"], x["eta"], x["beta"], x["gamma"], x["W"], x["M"], C, kind)
    W = [w[0].astype(np.float64) for w in x["W"]]
    for c in range(2):
        for t in range(C):
            assert rel(out["o"][0, c * C + t], oracle.net(W, x["q"][0, c * C + t].astype(np.float64), kind)) < 1e-13
        G = per_token_G(x, W, kind, C, start=c * C)
        # W <- W + sum_t eta_t G_t : one gradient step on the eta-weighted summed chunk loss
        W = [w + sum(float(x["eta"][0, c * C + t]) * G[t][i] for t in range(C)) for i, w in enumerate(W)]
        M_last = [float(x["eta"][0, c * C + C - 1]) * G[C - 1][i] for i in range(len(W))]
    for i in range(len(W)):
        assert rel(out["W"][i][0], W[i]) < 1e-12
        assert rel(out["M"][i][0], M_last[i]) < 1e-12


# ---------------------------------------------------------------- P7: hand-expanded C = 2
def test_two_token_chunk_matches_hand_expansion():
    coef = {}
    with open(os.path.join(GOLDEN, "c2_coefficients.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            name, *vals = line.split()
            coef[name] = [float(v) for v in vals]
    kind = oracle.KIND_MLP
    r, x = tiny(kind, L=2, C=2, seed=11)
    x["eta"][0] = [0.5, 0.25]
    x["beta"][:] = 0.5
    x["gamma"][:] = 0.5
    W0 = [w[0].astype(np.float64) for w in x["W"]]
    M0 = [m[0].astype(np.float64) for m in x["M"]]
    G = per_token_G(x, W0, kind, 2)
    out = oracle.forward(x["q"], x["k"], x["v"], x["eta"], x["beta"], x["gamma"], x["W"], x["M"], 2, kind)
    for i in range(2):
        cw, cm, c1, c2 = coef["W_2"]
        assert rel(out["W"][i][0], cw * W0[i] + cm * M0[i] + c1 * G[0][i] + c2 * G[1][i]) < 1e-13
        cw, cm, c1, c2 = coef["M_2"]
        assert rel(out["M"][i][0], cw * W0[i] + cm * M0[i] + c1 * G[0][i] + c2 * G[1][i]) < 1e-13


# ---------------------------------------------------------------- P10: split invariance, ragged tail
@pytest.mark.parametrize("kind", KINDS)
def test_split_calls_chain_bitwise(kind):
    r, x = tiny(kind, L=16, C=4, seed=13)
    full = oracle.forward(x["q"], x["k"], x["v"], x["eta"], x["beta"], x["gamma"], x["W"], x["M"], 4, kind,
                          want_states=True)
    a = oracle.forward(x["q"][:, :8], x["k"][:, :8], x["v"][:, :8], x["eta"][:, :8], x["beta"][:, :8],
                       x["gamma"][:, :8], x["W"], x["M"], 4, kind)
    b = oracle.forward(x["q"][:, 8:], x["k"][:, 8:], x["v"][:, 8:], x["eta"][:, 8:], x["beta"][:, 8:],
                       x["gamma"][:, 8:], a["W"], a["M"], 4, kind)
    assert np.array_equal(np.concatenate([a["o"], b["o"]], axis=1), full["o"])
    for i in range(len(x["W"])):
        assert np.array_equal(b["W"][i], full["W"][i]) and np.array_equal(b["M"][i], full["M"][i])
        # recorded chunk-start state of chunk 2 is the first call's final state
        assert np.array_equal(full["states"][0, 2, 0, i].reshape(a["W"][i][0].shape), a["W"][i][0])
        assert np.array_equal(full["states"][0, 2, 1, i].reshape(a["M"][i][0].shape), a["M"][i][0])


def test_ragged_tail_chunk_is_a_shorter_chunk():
    kind = oracle.KIND_MLP
    r, x = tiny(kind, L=10, C=4, seed=15)
    full = oracle.forward(x["q"], x["k"], x["v"], x["eta"], x["beta"], x["gamma"], x["W"], x["M"], 4, kind)
    a = oracle.forward(x["q"][:, :8], x["k"][:, :8], x["v"][:, :8], x["eta"][:, :8], x["beta"][:, :8],
                       x["gamma"][:, :8], x["W"], x["M"], 4, kind)
    b = oracle.forward(x["q"][:, 8:], x["k"][:, 8:], x["v"][:, 8:], x["eta"][:, 8:], x["beta"][:, 8:],
                       x["gamma"][:, 8:], a["W"], a["M"], 2, kind)
    assert np.array_equal(np.concatenate([a["o"], b["o"]], axis=1), full["o"])
    assert np.array_equal(b["W"][1], full["W"][1])


def test_sequences_are_independent_and_thread_count_does_not_matter():
    kind = oracle.KIND_MLP
    r, x = tiny(kind, L=8, C=4, seed=17, N=3)
    one = oracle.forward(x["q"], x["k"], x["v"], x["eta"], x["beta"], x["gamma"], x["W"], x["M"], 4, kind, threads=1)
    many = oracle.forward(x["q"], x["k"], x["v"], x["eta"], x["beta"], x["gamma"], x["W"], x["M"], 4, kind, threads=3)
    assert np.array_equal(one["o"], many["o"])
    solo = oracle.forward(x["q"][1:2], x["k"][1:2], x["v"][1:2], x["eta"][1:2], x["beta"][1:2], x["gamma"][1:2],
                          [w[1:2] for w in x["W"]], [m[1:2] for m in x["M"]], 4, kind)
    assert np.array_equal(solo["o"][0], one["o"][1])


# ---------------------------------------------------------------- P9: reverse pass vs autograd and finite differences
def torch_sequential(x, C, kind, eps=1e-5):
    """The same program by a different route: torch fp64, G_t from autograd (create_graph=True)."""
    F = torch.nn.functional
    T = lambda a: torch.tensor(np.asarray(a, dtype=np.float64), requires_grad=True)
    q, k, v = T(x["q"][0]), T(x["k"][0]), T(x["v"][0])
    eta, beta, gamma = T(x["eta"][0]), T(x["beta"][0]), T(x["gamma"][0])
    W_in = [T(w[0]) for w in x["W"]]
    M_in = [T(m[0]) for m in x["M"]]

    def f(W, xx):
        if kind == oracle.KIND_MLP:
            u = F.gelu(xx @ W[0].T) @ W[1].T
        else:
            u = (F.silu(xx @ W[0].T) * (xx @ W[1].T)) @ W[2].T
        return xx + F.layer_norm(u, (u.shape[-1],), eps=eps)

    W, M = list(W_in), list(M_in)
    L = q.shape[0]
    outs = []
    for s in range(0, L, C):
        W0 = list(W)
        outs.append(f(W0, q[s:s + C]))
        for t in range(s, min(s + C, L)):
            loss = 0.5 * ((f(W0, k[t]) - v[t]) ** 2).sum()
            g = torch.autograd.grad(loss, W0, create_graph=True)
            M = [beta[t] * m - eta[t] * gi for m, gi in zip(M, g)]
            W = [gamma[t] * w + m for w, m in zip(W, M)]
    o = torch.cat(outs, 0)
    leaves = dict(q=q, k=k, v=v, eta=eta, beta=beta, gamma=gamma, W=W_in, M=M_in)
    return o, W, M, leaves


@pytest.mark.parametrize("kind", KINDS)
def test_forward_and_reverse_match_independent_autograd(kind):
    C = 4
    r, x = tiny(kind, d=4, h=8, L=2 * C + 2, C=C, seed=19)  # two full chunks and a ragged tail
    o, Wf, Mf, lv = torch_sequential(x, C, kind)
    fw = oracle.forward(x["q"], x["k"], x["v"], x["eta"], x["beta"], x["gamma"], x["W"], x["M"], C, kind)
    assert rel(fw["o"][0], o.detach().numpy()) < 1e-12
    for i in range(len(Wf)):
        assert rel(fw["W"][i][0], Wf[i].detach().numpy()) < 1e-12
        assert rel(fw["M"][i][0], Mf[i].detach().numpy()) < 1e-12
    d_o = torch.tensor(x["d_o"][0], dtype=torch.float64)
    dW = [torch.tensor(a[0], dtype=torch.float64) for a in x["dW"]]
    dM = [torch.tensor(a[0], dtype=torch.float64) for a in x["dM"]]
    total = (o * d_o).sum() + sum((w * g).sum() for w, g in zip(Wf, dW)) + sum((m * g).sum() for m, g in zip(Mf, dM))
    flat = [lv["q"], lv["k"], lv["v"], lv["eta"], lv["beta"], lv["gamma"]] + lv["W"] + lv["M"]
    grads = torch.autograd.grad(total, flat)
    bw = oracle.backward(x["q"], x["k"], x["v"], x["eta"], x["beta"], x["gamma"], x["W"], x["M"],
                         x["d_o"], x["dW"], x["dM"], C, kind)
    names = ["dq", "dk", "dv", "deta", "dbeta", "dgamma"]
    for n, g in zip(names, grads[:6]):
        assert rel(bw[n][0], g.numpy()) < 1e-10, n
    nm = len(x["W"])
    for i in range(nm):
        assert rel(bw["dW"][i][0], grads[6 + i].numpy()) < 1e-10, ("dW", i)
        assert rel(bw["dM"][i][0], grads[6 + nm + i].numpy()) < 1e-10, ("dM", i)


@pytest.mark.parametrize("kind", KINDS)
def test_reverse_pass_matches_finite_differences_of_own_forward(kind):
    C = 4
    r, x = tiny(kind, d=4, h=8, L=2 * C, C=C, seed=23)
    bw = oracle.backward(x["q"], x["k"], x["v"], x["eta"], x["beta"], x["gamma"], x["W"], x["M"],
                         x["d_o"], x["dW"], x["dM"], C, kind)

    def objective(xx):
        fw = oracle.forward(xx["q"], xx["k"], xx["v"], xx["eta"], xx["beta"], xx["gamma"], xx["W"], xx["M"], C, kind)
        s = float(np.sum(fw["o"] * xx["d_o"]))
        for i in range(len(xx["W"])):
            s += float(np.sum(fw["W"][i] * xx["dW"][i]) + np.sum(fw["M"][i] * xx["dM"][i]))
        return s

    x64 = {n: (([a.astype(np.float64) for a in val]) if isinstance(val, list) else val.astype(np.float64))
           for n, val in x.items()}
    rng = np.random.default_rng(0)
    step = 1e-6
    probes = [("q", "dq"), ("k", "dk"), ("v", "dv"), ("eta", "deta"), ("beta", "dbeta"), ("gamma", "dgamma")]
    for name, gname in probes:
        for _ in range(4):
            idx = tuple(rng.integers(0, s) for s in x64[name].shape)
            keep = x64[name][idx]
            x64[name][idx] = keep + step
            up = objective(x64)
            x64[name][idx] = keep - step
            dn = objective(x64)
            x64[name][idx] = keep
            fd = (up - dn) / (2 * step)
            assert abs(fd - bw[gname][idx]) <= 2e-6 * max(1.0, abs(fd)), (name, idx, fd, bw[gname][idx])
    for name, gname in (("W", "dW"), ("M", "dM")):
        for i in range(len(x64[name])):
            for _ in range(3):
                idx = tuple(rng.integers(0, s) for s in x64[name][i].shape)
                keep = x64[name][i][idx]
                x64[name][i][idx] = keep + step
                up = objective(x64)
                x64[name][i][idx] = keep - step
                dn = objective(x64)
                x64[name][i][idx] = keep
                fd = (up - dn) / (2 * step)
                assert abs(fd - bw[gname][i][idx]) <= 2e-6 * max(1.0, abs(fd)), (name, i, idx, fd, bw[gname][i][idx])



# ---------------------------------------------------------------- post-chunk normalisation (a reading: rows, to a target)
def _targets(x, scale=1.0):
    """Target norms as a model would set them: the row norms of the initial fast weights (times a factor)."""
    return [scale * np.sqrt((w.astype(np.float64) ** 2).sum(-1)) for w in x["W"]]


def _normalise_rows(W, target, eps_n):
    """Independent restatement in numpy: every row w -> n w / (||w|| + eps_n)."""
    s = np.sqrt((W ** 2).sum(-1, keepdims=True))
    return W * (target[..., None] / (s + eps_n))


@pytest.mark.parametrize("kind", KINDS)
def test_post_chunk_normalisation_equals_chunk_by_chunk_restatement(kind):
    """Normalised run == for every chunk: the (already pinned) un-normalised update of that chunk alone, followed by a
    row normalisation written here in numpy.  Also: the final rows have norm n s/(s + eps_n), the momentum is untouched
    by the normalisation itself, and the outputs of chunk c come from the normalised state of chunk c - 1."""
    C, eps_n = 4, 1e-5
    r, x = tiny(kind, d=4, h=8, L=3 * C + 2, C=C, seed=31, N=2)
    tgt = _targets(x, 1.3)
    got = oracle.forward(x["q"], x["k"], x["v"], x["eta"], x["beta"], x["gamma"], x["W"], x["M"], C, kind,
                         row_norm=tgt, norm_eps=eps_n)
    W = [w.astype(np.float64) for w in x["W"]]
    M = [m.astype(np.float64) for m in x["M"]]
    outs = []
    for s0 in range(0, r.L, C):
        sl = slice(s0, min(s0 + C, r.L))
        one = oracle.forward(x["q"][:, sl], x["k"][:, sl], x["v"][:, sl], x["eta"][:, sl], x["beta"][:, sl],
                             x["gamma"][:, sl], W, M, C, kind)
        outs.append(one["o"])
        pre = one["W"]
        W = [_normalise_rows(w, t, eps_n) for w, t in zip(pre, tgt)]
        M = one["M"]
    assert rel(got["o"], np.concatenate(outs, 1)) <= 1e-13
    for i in range(len(W)):
        assert rel(got["W"][i], W[i]) <= 1e-13 and rel(got["M"][i], M[i]) <= 1e-13
        s_pre = np.sqrt((pre[i] ** 2).sum(-1))
        assert np.allclose(np.sqrt((got["W"][i] ** 2).sum(-1)), tgt[i] * s_pre / (s_pre + eps_n), rtol=1e-12)
    plain = oracle.forward(x["q"], x["k"], x["v"], x["eta"], x["beta"], x["gamma"], x["W"], x["M"], C, kind)
    assert rel(got["o"][:, :C], plain["o"][:, :C]) == 0.0           # the first chunk reads the un-normalised initial state
    assert rel(got["o"][:, C:], plain["o"][:, C:]) > 1e-3           # later chunks do see the normalisation


def test_post_chunk_normalisation_is_invariant_to_the_scale_of_the_update():
    """Rows that are rescaled to a fixed norm forget their length: with targets t, a run started from c * W_init
    (eta = 0, gamma = 1, so the update leaves the direction alone) ends at rows of norm t in the direction of W_init."""
    C, eps_n = 4, 0.0
    r, x = tiny(inputs.KIND_MLP, d=4, h=8, L=2 * C, C=C, seed=33, m_std=0.0)
    x["eta"][:] = 0.0
    x["gamma"][:] = 1.0
    tgt = [np.full(w.shape[:2], 2.0) for w in x["W"]]
    got = oracle.forward(x["q"], x["k"], x["v"], x["eta"], x["beta"], x["gamma"], [5.0 * w.astype(np.float64) for w in x["W"]], x["M"], C, inputs.KIND_MLP,
                         row_norm=tgt, norm_eps=eps_n)
    for i, w in enumerate(x["W"]):
        w = w.astype(np.float64)
        unit = w / np.sqrt((w ** 2).sum(-1, keepdims=True))
        assert rel(got["W"][i], 2.0 * unit) <= 1e-13


@pytest.mark.parametrize("kind", KINDS)
def test_reverse_pass_through_the_normalisation_matches_finite_differences(kind):
    C, eps_n = 3, 1e-3
    r, x = tiny(kind, d=4, h=6, L=2 * C + 1, C=C, seed=37)
    x64 = {n: (([a.astype(np.float64) for a in val]) if isinstance(val, list) else val.astype(np.float64))
           for n, val in x.items()}
    x64["row_norm"] = _targets(x, 0.8)
    bw = oracle.backward(x64["q"], x64["k"], x64["v"], x64["eta"], x64["beta"], x64["gamma"], x64["W"], x64["M"],
                         x64["d_o"], x64["dW"], x64["dM"], C, kind, row_norm=x64["row_norm"], norm_eps=eps_n)

    def objective(xx):
        fw = oracle.forward(xx["q"], xx["k"], xx["v"], xx["eta"], xx["beta"], xx["gamma"], xx["W"], xx["M"], C, kind,
                            row_norm=xx["row_norm"], norm_eps=eps_n)
        s = float(np.sum(fw["o"] * xx["d_o"]))
        for i in range(len(xx["W"])):
            s += float(np.sum(fw["W"][i] * xx["dW"][i]) + np.sum(fw["M"][i] * xx["dM"][i]))
        return s

    rng = np.random.default_rng(1)
    step = 1e-6

    def probe(arr, grad, what):
        idx = tuple(rng.integers(0, s) for s in arr.shape)
        keep = arr[idx]
        arr[idx] = keep + step
        up = objective(x64)
        arr[idx] = keep - step
        dn = objective(x64)
        arr[idx] = keep
        fd = (up - dn) / (2 * step)
        assert abs(fd - grad[idx]) <= 5e-6 * max(1.0, abs(fd)), (what, idx, fd, grad[idx])

    for name, gname in [("q", "dq"), ("k", "dk"), ("v", "dv"), ("eta", "deta"), ("beta", "dbeta"), ("gamma", "dgamma")]:
        for _ in range(4):
            probe(x64[name], bw[gname], name)
    for name, gname in (("W", "dW"), ("M", "dM"), ("row_norm", "drow_norm")):
        for i in range(len(x64[name])):
            for _ in range(3):
                probe(x64[name][i], bw[gname][i], (name, i))
    # without normalisation the new entry points are the old ones
    a = oracle.backward(x64["q"], x64["k"], x64["v"], x64["eta"], x64["beta"], x64["gamma"], x64["W"], x64["M"],
                        x64["d_o"], x64["dW"], x64["dM"], C, kind)
    assert "drow_norm" not in a


# ---------------------------------------------------------------- input generator sanity (data only)
def test_generator_follows_the_stated_distributions():
    r = inputs.config(0)
    x = inputs.generate(r)
    assert np.allclose(np.linalg.norm(x["k"].astype(np.float64), axis=-1), 1.0, atol=1e-6)
    assert 0 < x["eta"].min() and x["eta"].max() < 0.1
    assert 0.9 < x["gamma"].min() and x["gamma"].max() < 1.0      # gamma = 1 - eta * alpha
    assert abs(float(x["W"][0].std()) - 0.02) < 2e-3
    r1 = inputs.config(1, heads=[5])
    a = inputs.generate(r1)
    b = inputs.generate(inputs.config(1, heads=[4, 5]))
    assert np.array_equal(a["q"][0], b["q"][1])                    # a head alone == the same head in a batch
    bits = inputs.to_bf16_bits(a["q"])
    assert np.array_equal(inputs.from_bf16_bits(bits), a["q"])     # bf16 I/O values are exactly representable
    t = torch.tensor(inputs.generate(inputs.config(1, heads=[5], io="f32"))["q"])
    assert np.array_equal(t.to(torch.bfloat16).float().numpy(), a["q"])  # same rounding as the hardware convert


# ---------------------------------------------------------------- token preparation (SiLU + L2 norm, gate parameterisation)
def test_prepare_oracle_matches_library_ops_and_autograd():
    from oracle import prepare
    rng = np.random.default_rng(3)
    x = rng.standard_normal((5, 7, 16))
    yb = rng.standard_normal((5, 7, 16))
    xt = torch.tensor(x, dtype=torch.float64, requires_grad=True)
    yt = torch.nn.functional.normalize(torch.nn.functional.silu(xt), dim=-1, eps=1e-12)
    assert rel(prepare.silu_l2norm(x), yt.detach().numpy()) <= 1e-14
    (yt * torch.tensor(yb)).sum().backward()
    assert rel(prepare.silu_l2norm_vjp(x, yb), xt.grad.numpy()) <= 1e-12
    assert np.allclose(np.sqrt((prepare.silu_l2norm(x) ** 2).sum(-1)), 1.0, atol=1e-14)       # unit rows
    assert np.array_equal(prepare.silu_l2norm(np.zeros((2, 4))), np.zeros((2, 4)))            # zero vector stays zero
    a, b, c = (rng.standard_normal((5, 7)) * 2 for _ in range(3))
    de, db, dg = (rng.standard_normal((5, 7)) for _ in range(3))
    eb, tau, ab = 0.01, 32.0, 0.1
    at, bt, ct = (torch.tensor(t, dtype=torch.float64, requires_grad=True) for t in (a, b, c))
    eta_t = eb * torch.sigmoid(at)
    beta_t = torch.sigmoid(bt) ** (1.0 / tau)
    gamma_t = 1.0 - eta_t * (ab * torch.sigmoid(ct))
    eta, beta, gamma = prepare.gates(a, b, c, eb, tau, ab)
    assert rel(eta, eta_t.detach().numpy()) <= 1e-14 and rel(beta, beta_t.detach().numpy()) <= 1e-14
    assert rel(gamma, gamma_t.detach().numpy()) <= 1e-14
    (eta_t * torch.tensor(de) + beta_t * torch.tensor(db) + gamma_t * torch.tensor(dg)).sum().backward()
    da, dbb, dc = prepare.gates_vjp(a, b, c, eb, tau, ab, de, db, dg)
    assert rel(da, at.grad.numpy()) <= 1e-12 and rel(dbb, bt.grad.numpy()) <= 1e-12 and rel(dc, ct.grad.numpy()) <= 1e-12
    # ranges the method relies on: 0 < eta < eta_base, 0 < beta < 1, 1 - eta_base alpha_base < gamma < 1
    assert (eta > 0).all() and (eta < eb).all() and (beta > 0).all() and (beta < 1).all()
    assert (gamma < 1).all() and (gamma > 1 - eb * ab).all()


# ------------------------------------------------------------------ matrix form of the chunk (oracle/chunk_form.py)
def test_chunk_matrix_form_equals_the_sequential_oracle():
    """Algorithm 1 in matrix form (one inner forward/backward at the chunk-start weights, scalar kernels, Proposition 1)
    against the token-by-token program, four chunks free-running: a pin of both (different language, different
    formulation, same numbers)."""
    from oracle import chunk_form
    r = inputs.Recipe(B=1, H=2, L=28, d=8, h=16, C=8, kind=inputs.KIND_MLP, io="f32", seed=11, m_std=0.05, w_std=0.3)   # ragged last chunk
    x = inputs.generate(r)
    ref = oracle.forward(x["q"], x["k"], x["v"], x["eta"], x["beta"], x["gamma"], x["W"], x["M"], r.C, r.kind)
    for n in range(2):
        o, (W1, W2, M1, M2) = chunk_form.forward_mlp(x["q"][n], x["k"][n], x["v"][n], x["eta"][n], x["beta"][n], x["gamma"][n],
                                                     x["W"][0][n], x["W"][1][n], x["M"][0][n], x["M"][1][n], r.C)
        assert np.max(np.abs(o - ref["o"][n])) < 1e-10
        for got, want in ((W1, ref["W"][0][n]), (W2, ref["W"][1][n]), (M1, ref["M"][0][n]), (M2, ref["M"][1][n])):
            assert np.max(np.abs(got - want)) < 1e-10 * max(1.0, np.max(np.abs(want)))


def test_closed_form_in_fp32_tracks_the_sequential_recurrence_in_fp32():
    """The paper's numerical-equivalence experiment (Section 3.2; Appendix "Exactness"): closed form and token-wise
    recurrence, both in fp32, over many chunks of 512 tokens under the paper's gate regime, stay at a relative l2
    deviation of order 1e-6 in W_C and M_C (the paper reports < 2e-6 over 128 chunks).  Synthetic inputs, 16 chunks,
    small d.  Two readings are checked: every chunk from the same start state (the two evaluations of one chunk), and
    two free-running fp32 chains (where the map's own sensitivity adds to the rounding)."""
    from oracle import chunk_form
    r = inputs.paper_regime(inputs.Recipe(B=1, H=1, L=16 * 512, d=16, h=32, C=512, kind=inputs.KIND_MLP, io="f32", seed=5, m_std=0.002))
    x = inputs.generate(r)
    f32 = np.float32
    q, k, v, eta, beta, gamma = (x[n][0] for n in ("q", "k", "v", "eta", "beta", "gamma"))
    a = tuple(m[0].astype(f32) for m in (x["W"][0], x["W"][1], x["M"][0], x["M"][1]))   # closed-form chain
    b = a                                                                                 # sequential chain

    def rel(x_, y_):
        return float(np.linalg.norm(x_.astype(np.float64) - y_.astype(np.float64)) / np.linalg.norm(y_.astype(np.float64)))

    def sequential_chunk(state, sl):
        _, _, pc = chunk_form.chunk_mlp(k[sl], q[sl], v[sl], eta[sl], beta[sl], gamma[sl], *state, dtype=f32)
        G2 = [-np.outer(pc["Pu"][t], pc["A"][t]) for t in range(r.C)]
        G1 = [-np.outer(pc["Pz"][t], k[sl][t].astype(f32)) for t in range(r.C)]
        W1s, M1s = chunk_form.sequential_from_grads(state[0], state[2], G1, eta[sl], beta[sl], gamma[sl], f32)
        W2s, M2s = chunk_form.sequential_from_grads(state[1], state[3], G2, eta[sl], beta[sl], gamma[sl], f32)
        return (W1s, W2s, M1s, M2s)

    worst_chunk = 0.0
    for s in range(0, r.L, r.C):
        sl = slice(s, s + r.C)
        same_start = sequential_chunk(a, sl)
        _, a, _ = chunk_form.chunk_mlp(k[sl], q[sl], v[sl], eta[sl], beta[sl], gamma[sl], *a, dtype=f32)
        worst_chunk = max(worst_chunk, max(rel(x_, y_) for x_, y_ in zip(a, same_start)))
        b = sequential_chunk(b, sl)
    free = max(rel(x_, y_) for x_, y_ in zip(a, b))
    print(f"fp32 closed form vs fp32 sequential, 16 chunks of 512: worst single chunk {worst_chunk:.2e}, free-running chains {free:.2e}")
    assert worst_chunk < 3e-6
    assert free < 5e-5


def test_rounding_hooks_move_the_result_by_a_bf16_amount_and_nothing_else():
    """Hooked mode = the same fp64 program with bf16 roundings at the declared points: it must stay within a few bf16
    ulps of the unhooked result (and must differ from it)."""
    from oracle import chunk_form
    r = inputs.Recipe(B=1, H=1, L=64, d=32, h=64, C=64, kind=inputs.KIND_MLP, io="bf16", seed=2, m_std=0.002)
    x = inputs.generate(r)
    args = [x[n][0] for n in ("q", "k", "v", "eta", "beta", "gamma")] + [x["W"][0][0], x["W"][1][0], x["M"][0][0], x["M"][1][0], r.C]
    o0, s0 = chunk_form.forward_mlp(*args)
    o1, s1 = chunk_form.forward_mlp(*args, hooks=chunk_form.Hooks(gelu="erf"))
    for got, want in [(o1, o0)] + list(zip(s1, s0)):
        e = np.max(np.abs(got - want)) / np.max(np.abs(want))
        assert 1e-5 < e < 2e-2, e
