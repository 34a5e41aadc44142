"""Post-chunk normalisation of the fast weights (e2ttt_chunk_fwd_normed / e2ttt_chunk_bwd_normed) against the oracle."""
import numpy as np
import pytest
import torch

from paper_2608_21308_b200 import binding as E
from paper_2608_21308_b200 import inputs
from tests import util
from tests.test_gpu_parity import TOL_BF16, TOL_F32, check_backward, check_forward

pytestmark = pytest.mark.gpu
MLP, SWIGLU = inputs.KIND_MLP, inputs.KIND_SWIGLU
EPS_N = 1e-5


def targets(x, scale=1.0):
    return [(scale * np.sqrt((w.astype(np.float64) ** 2).sum(-1))).astype(np.float32) for w in x["W"]]


def _dev(a, dtype=torch.float32):
    return torch.tensor(np.ascontiguousarray(a), dtype=torch.float32).to(dtype).cuda().contiguous()


def gpu_forward_normed(x, tgt, *, d, h, C, kind, io, impl, save_states=False, norm_eps=EPS_N):
    N, L, _ = x["q"].shape
    p = E.make_params(N, 1, L, d, h, C, kind, E.E2TTT_F32 if io == "f32" else E.E2TTT_BF16, 1e-5, impl)
    iod = torch.float32 if io == "f32" else torch.bfloat16
    q, k, v = (_dev(x[n], iod).view(N, 1, L, d) for n in ("q", "k", "v"))
    eta, beta, gamma = (_dev(x[n]).view(N, 1, L) for n in ("eta", "beta", "gamma"))
    W = [_dev(w).unsqueeze(1).contiguous() for w in x["W"]]
    M = [_dev(m).unsqueeze(1).contiguous() for m in x["M"]]
    rn = [_dev(t).unsqueeze(1).contiguous() for t in tgt]
    o = torch.empty_like(q)
    Wf = [torch.empty_like(w) for w in W]
    Mf = [torch.empty_like(w) for w in W]
    ws = torch.empty(E.e2ttt_workspace_bytes_normed(p, int(save_states)), dtype=torch.uint8, device="cuda")
    E.e2ttt_chunk_fwd_normed(p, q, k, v, eta, beta, gamma, W, M, rn, norm_eps, o, Wf, Mf, ws, int(save_states))
    torch.cuda.synchronize()
    assert E.e2ttt_device_status(ws) == 0
    return {"o": o.float().cpu().numpy().reshape(N, L, d), "W": [w.cpu().numpy()[:, 0] for w in Wf],
            "M": [m.cpu().numpy()[:, 0] for m in Mf]}


def gpu_backward_normed(x, tgt, *, d, h, C, kind, io, impl, via_saved_states):
    N, L, _ = x["q"].shape
    p = E.make_params(N, 1, L, d, h, C, kind, E.E2TTT_F32 if io == "f32" else E.E2TTT_BF16, 1e-5, impl)
    iod = torch.float32 if io == "f32" else torch.bfloat16
    q, k, v, d_o = (_dev(x[n], iod).view(N, 1, L, d) for n in ("q", "k", "v", "d_o"))
    eta, beta, gamma = (_dev(x[n]).view(N, 1, L) for n in ("eta", "beta", "gamma"))
    W = [_dev(w).unsqueeze(1).contiguous() for w in x["W"]]
    M = [_dev(m).unsqueeze(1).contiguous() for m in x["M"]]
    dWf = [_dev(w).unsqueeze(1).contiguous() for w in x["dW"]]
    dMf = [_dev(w).unsqueeze(1).contiguous() for w in x["dM"]]
    rn = [_dev(t).unsqueeze(1).contiguous() for t in tgt]
    drn = [torch.full_like(t, float("nan")) for t in rn]
    dq, dk, dv = torch.empty_like(q), torch.empty_like(q), torch.empty_like(q)
    de, db, dg = torch.empty_like(eta), torch.empty_like(eta), torch.empty_like(eta)
    dW = [torch.empty_like(w) for w in W]
    dM = [torch.empty_like(w) for w in W]
    ws = torch.empty(E.e2ttt_workspace_bytes_normed(p, 1), dtype=torch.uint8, device="cuda")
    if via_saved_states:
        o = torch.empty_like(q)
        Wf = [torch.empty_like(w) for w in W]
        Mf = [torch.empty_like(w) for w in W]
        E.e2ttt_chunk_fwd_normed(p, q, k, v, eta, beta, gamma, W, M, rn, EPS_N, o, Wf, Mf, ws, 1)
    E.e2ttt_chunk_bwd_normed(p, q, k, v, eta, beta, gamma, W, M, rn, EPS_N, d_o, dWf, dMf, dq, dk, dv, de, db, dg, dW, dM,
                             drn, ws, int(via_saved_states))
    torch.cuda.synchronize()
    assert E.e2ttt_device_status(ws) == 0
    f = lambda t: t.float().cpu().numpy()
    return {"dq": f(dq).reshape(N, L, d), "dk": f(dk).reshape(N, L, d), "dv": f(dv).reshape(N, L, d),
            "deta": f(de).reshape(N, L), "dbeta": f(db).reshape(N, L), "dgamma": f(dg).reshape(N, L),
            "dW": [f(w)[:, 0] for w in dW], "dM": [f(m)[:, 0] for m in dM], "drow_norm": [f(t)[:, 0] for t in drn]}


def oracle_fwd(x, tgt, C, kind):
    from oracle import oracle
    return oracle.forward(x["q"], x["k"], x["v"], x["eta"], x["beta"], x["gamma"], x["W"], x["M"], C, kind,
                          row_norm=tgt, norm_eps=EPS_N)


def oracle_bwd(x, tgt, C, kind):
    from oracle import oracle
    return oracle.backward(x["q"], x["k"], x["v"], x["eta"], x["beta"], x["gamma"], x["W"], x["M"], x["d_o"], x["dW"],
                           x["dM"], C, kind, row_norm=tgt, norm_eps=EPS_N)


@pytest.mark.parametrize("kind", [MLP, SWIGLU])
@pytest.mark.parametrize("d,h,C,L,N", [(48, 80, 24, 100, 3), (64, 256, 16, 64, 2), (8, 16, 1, 5, 1)])
def test_normed_forward_free_running_fp32(kind, d, h, C, L, N):
    r = inputs.paper_regime(inputs.Recipe(B=N, H=1, L=L, d=d, h=h, C=C, kind=kind, io="f32", seed=41, m_std=0.002))
    x = inputs.generate(r)
    tgt = targets(x, 1.2)
    ref = oracle_fwd(x, tgt, C, kind)
    got = gpu_forward_normed(x, tgt, d=d, h=h, C=C, kind=kind, io="f32", impl=E.E2TTT_IMPL_AUTO)
    check_forward(got, ref, TOL_F32, "normed fwd fp32")
    for i, t in enumerate(tgt):   # the property itself: rows end at their target norm (up to eps_n)
        assert np.allclose(np.sqrt((got["W"][i].astype(np.float64) ** 2).sum(-1)), t, rtol=1e-3)


@pytest.mark.parametrize("impl", [E.E2TTT_IMPL_TILED, E.E2TTT_IMPL_SIMT, E.E2TTT_IMPL_AUTO], ids=["tiled", "simt", "auto"])
@pytest.mark.parametrize("cfg", [2, 3])
def test_normed_forward_windows_bf16(cfg, impl):
    """Benchmark shapes (config 2's shape has a fused kernel, which does not normalise: AUTO must not pick it)."""
    r = inputs.config(cfg, heads=[3, 30], m_std=0.002)
    xw, _ = util.teacher_forced_windows(r, 3, window=1)
    tgt = targets(xw, 0.9)
    ref = oracle_fwd(xw, tgt, r.C, r.kind)
    got = gpu_forward_normed(xw, tgt, d=r.d, h=r.h, C=r.C, kind=r.kind, io="bf16", impl=impl)
    check_forward(got, ref, TOL_BF16, f"normed fwd bf16 config {cfg}")


@pytest.mark.parametrize("kind", [MLP, SWIGLU])
@pytest.mark.parametrize("saved", [False, True])
def test_normed_backward_free_running_fp32(kind, saved):
    r = inputs.paper_regime(inputs.Recipe(B=2, H=1, L=60, d=48, h=80, C=24, kind=kind, io="f32", seed=43, m_std=0.002))
    x = inputs.generate(r, with_d_o=True, with_dstate=True)
    tgt = targets(x, 1.1)
    ref = oracle_bwd(x, tgt, r.C, kind)
    got = gpu_backward_normed(x, tgt, d=r.d, h=r.h, C=r.C, kind=kind, io="f32", impl=E.E2TTT_IMPL_AUTO,
                              via_saved_states=saved)
    check_backward(got, ref, TOL_F32, "normed bwd fp32")
    for i in range(len(tgt)):
        assert util.rel_err(got["drow_norm"][i], ref["drow_norm"][i]) <= TOL_F32, i


@pytest.mark.parametrize("cfg", [4, 3])
def test_normed_backward_windows_bf16(cfg):
    r = inputs.config(cfg, heads=[2, 11])
    xw, _ = util.teacher_forced_windows(r, 3, window=1, with_grads=True)
    tgt = targets(xw, 1.0)
    ref = oracle_bwd(xw, tgt, r.C, r.kind)
    got = gpu_backward_normed(xw, tgt, d=r.d, h=r.h, C=r.C, kind=r.kind, io="bf16", impl=E.E2TTT_IMPL_AUTO,
                              via_saved_states=True)
    check_backward(got, ref, TOL_BF16, f"normed bwd bf16 config {cfg}")
    for i in range(len(tgt)):
        assert util.rel_err(got["drow_norm"][i], ref["drow_norm"][i]) <= TOL_BF16, i


def test_normed_calls_reject_missing_targets():
    r = inputs.config(2, heads=[0], L=64)
    x = inputs.generate(r)
    tgt = targets(x)
    with pytest.raises(Exception):
        gpu_forward_normed(x, tgt[:1], d=r.d, h=r.h, C=r.C, kind=r.kind, io="bf16", impl=E.E2TTT_IMPL_TILED)


# ---- the fused tensor-core forward with the normalisation in its state pass

@pytest.mark.parametrize("cfg,over", [(2, {}), (1, {}), (2, dict(h=384))], ids=["128x512", "64x256-padded", "128x384-padded"])
def test_fused_normed_forward_windows(cfg, over):
    r = inputs.config(cfg, heads=[3, 30], m_std=0.002, **over)
    xw, _ = util.teacher_forced_windows(r, 4, window=1)
    tgt = targets(xw, 0.9)
    ref = oracle_fwd(xw, tgt, r.C, r.kind)
    got = gpu_forward_normed(xw, tgt, d=r.d, h=r.h, C=r.C, kind=r.kind, io="bf16", impl=E.E2TTT_IMPL_TCGEN05)
    errs = check_forward(got, ref, TOL_BF16, f"fused normed fwd config {cfg} {over}")
    for i, t in enumerate(tgt):
        assert np.allclose(np.sqrt((got["W"][i].astype(np.float64) ** 2).sum(-1)), t, rtol=1e-3)
    print(errs)


@pytest.mark.parametrize("cfg,over", [(1, {}), (2, dict(h=384))], ids=["64x256-padded", "128x384-padded"])
def test_fused_normed_padded_shapes_with_zero_norm_eps(cfg, over):
    """norm_eps = 0 is allowed.  The padded rows of the 128 x 512 tiles have target 0 and norm 0: they must stay exactly
    0 (not 0/0), so every result is finite and agrees with the any-shape kernels."""
    r = inputs.config(cfg, heads=[3, 30], m_std=0.002, **over)
    xw, _ = util.teacher_forced_windows(r, 4, window=2)
    tgt = targets(xw, 0.9)
    shape = dict(d=r.d, h=r.h, C=r.C, kind=r.kind, io="bf16")
    fused = gpu_forward_normed(xw, tgt, impl=E.E2TTT_IMPL_TCGEN05, norm_eps=0.0, **shape)
    tiled = gpu_forward_normed(xw, tgt, impl=E.E2TTT_IMPL_TILED, norm_eps=0.0, **shape)
    assert np.isfinite(fused["o"]).all() and all(np.isfinite(w).all() for w in fused["W"] + fused["M"])
    assert util.rel_err(fused["o"], tiled["o"]) <= 3 * TOL_BF16
    for i in range(2):
        assert util.rel_err(fused["W"][i], tiled["W"][i]) <= 3 * TOL_BF16
        assert util.rel_err(fused["M"][i], tiled["M"][i]) <= 3 * TOL_BF16


def test_fused_normed_forward_free_running_and_auto_selection():
    """16 chunks free-running under the paper's gate regime; AUTO must take the fused kernel (same bits as TCGEN05);
    two calls of half the length chain to the same result (the final state is the normalised one)."""
    r = inputs.paper_regime(inputs.Recipe(B=3, H=1, L=1024, d=128, h=512, C=64, kind=MLP, io="bf16", seed=4, m_std=0.002))
    x = inputs.generate(r)
    tgt = targets(x, 1.1)
    ref = oracle_fwd(x, tgt, 64, MLP)
    shape = dict(d=128, h=512, C=64, kind=MLP, io="bf16")
    got = gpu_forward_normed(x, tgt, impl=E.E2TTT_IMPL_TCGEN05, **shape)
    check_forward(got, ref, TOL_BF16, "fused normed, 16 chunks free-running")
    auto = gpu_forward_normed(x, tgt, impl=E.E2TTT_IMPL_AUTO, **shape)
    assert np.array_equal(auto["o"], got["o"]) and all(np.array_equal(a, b) for a, b in zip(auto["W"], got["W"]))
    tiled = gpu_forward_normed(x, tgt, impl=E.E2TTT_IMPL_TILED, **shape)
    check_forward(tiled, ref, TOL_BF16, "tiled normed")
    half = r.L // 2
    first = {n: (np.ascontiguousarray(v[:, :half]) if not isinstance(v, list) else v) for n, v in x.items()}
    a = gpu_forward_normed(first, tgt, impl=E.E2TTT_IMPL_TCGEN05, **shape)
    rest = {n: (np.ascontiguousarray(v[:, half:]) if not isinstance(v, list) else v) for n, v in x.items()}
    rest["W"], rest["M"] = a["W"], a["M"]
    b = gpu_forward_normed(rest, tgt, impl=E.E2TTT_IMPL_TCGEN05, **shape)
    assert np.array_equal(np.concatenate([a["o"], b["o"]], 1), got["o"])
    for i in range(2):
        assert np.array_equal(b["W"][i], got["W"][i]) and np.array_equal(b["M"][i], got["M"][i])


def test_fused_normed_forward_saves_what_the_normalised_reverse_pass_reads():
    """Training flow: the fused forward (two chunks per call) writes start states, row norms and the final slot; the
    reverse pass from them agrees with the reverse pass that recomputes everything on the any-shape kernels, and a
    one-chunk window agrees with the oracle."""
    r = inputs.config(4, heads=[2, 11])
    x2, _ = util.teacher_forced_windows(r, 4, window=2, with_grads=True)
    tgt = targets(x2, 1.0)
    shape = dict(d=r.d, h=r.h, C=r.C, kind=r.kind, io="bf16")
    a = gpu_backward_normed(x2, tgt, impl=E.E2TTT_IMPL_TCGEN05, via_saved_states=True, **shape)
    b = gpu_backward_normed(x2, tgt, impl=E.E2TTT_IMPL_TILED, via_saved_states=False, **shape)
    for n in ("dq", "dk", "dv", "deta", "dbeta", "dgamma"):
        assert util.rel_err(a[n], b[n]) <= 3 * TOL_BF16, n
    for i in range(2):
        assert util.rel_err(a["drow_norm"][i], b["drow_norm"][i]) <= 3 * TOL_BF16, i
    x1, _ = util.teacher_forced_windows(r, 3, window=1, with_grads=True)
    tgt1 = targets(x1, 1.0)
    ref = oracle_bwd(x1, tgt1, r.C, r.kind)
    got = gpu_backward_normed(x1, tgt1, impl=E.E2TTT_IMPL_TCGEN05, via_saved_states=True, **shape)
    check_backward(got, ref, TOL_BF16, "normed bwd from the fused forward's saved states")
    for i in range(2):
        assert util.rel_err(got["drow_norm"][i], ref["drow_norm"][i]) <= TOL_BF16, i
