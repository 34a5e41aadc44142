"""Token preparation (SiLU + L2 normalisation of q and k, gate parameterisation) against its numpy oracle."""
import numpy as np
import pytest
import torch

from oracle import prepare as O
from paper_2608_21308_b200 import binding as E
from paper_2608_21308_b200 import inputs
from tests import util

pytestmark = pytest.mark.gpu
GP = dict(eta_base=0.01, tau=32.0, alpha_base=0.1, norm_eps=1e-12)


def _bf16(a):
    return inputs.round_bf16(a)


def _run(B, H, L, d, io, seed=0, backward=False):
    rng = np.random.default_rng(seed)
    rnd = _bf16 if io == "bf16" else (lambda a: a.astype(np.float32))
    x = {n: rnd(rng.standard_normal((B, H, L, d)).astype(np.float32)) for n in ("q_raw", "k_raw", "dq", "dk")}
    s = {n: (2.0 * rng.standard_normal((B, H, L))).astype(np.float32) for n in ("a_eta", "a_beta", "a_alpha")}
    g = {n: rng.standard_normal((B, H, L)).astype(np.float32) for n in ("d_eta", "d_beta", "d_gamma")}
    iod = torch.float32 if io == "f32" else torch.bfloat16
    p = E.make_params(B, H, L, d, 4 * d, 1, inputs.KIND_MLP, E.E2TTT_F32 if io == "f32" else E.E2TTT_BF16, 1e-5, E.E2TTT_IMPL_AUTO)
    gp = E.e2ttt_gate_params(GP["eta_base"], GP["tau"], GP["alpha_base"], GP["norm_eps"])
    dev = lambda a, t=torch.float32: torch.tensor(a, dtype=torch.float32).to(t).cuda().contiguous()
    qr, kr = dev(x["q_raw"], iod), dev(x["k_raw"], iod)
    ae, ab, aa = dev(s["a_eta"]), dev(s["a_beta"]), dev(s["a_alpha"])
    out = {}
    if not backward:
        q, k = torch.empty_like(qr), torch.empty_like(kr)
        eta, beta, gamma = torch.empty_like(ae), torch.empty_like(ae), torch.empty_like(ae)
        E.e2ttt_prepare_fwd(p, gp, qr, kr, ae, ab, aa, q, k, eta, beta, gamma)
        torch.cuda.synchronize()
        out = {"q": q, "k": k, "eta": eta, "beta": beta, "gamma": gamma}
    else:
        dq, dk = dev(x["dq"], iod), dev(x["dk"], iod)
        de, db, dg = dev(g["d_eta"]), dev(g["d_beta"]), dev(g["d_gamma"])
        dqr, dkr = torch.empty_like(qr), torch.empty_like(kr)
        dae, dab, daa = torch.empty_like(ae), torch.empty_like(ae), torch.empty_like(ae)
        E.e2ttt_prepare_bwd(p, gp, qr, kr, ae, ab, aa, dq, dk, de, db, dg, dqr, dkr, dae, dab, daa)
        torch.cuda.synchronize()
        out = {"dq_raw": dqr, "dk_raw": dkr, "da_eta": dae, "da_beta": dab, "da_alpha": daa}
    return x, s, g, {n: t.float().cpu().numpy() for n, t in out.items()}


SHAPES = [(2, 3, 17, 128), (1, 2, 5, 64), (1, 1, 3, 48), (2, 1, 7, 256), (1, 1, 2, 1000), (1, 1, 1, 8), (1, 2, 33, 130),
          # the bulk-copy pipeline of the forward: several tiles per CTA, a ragged last tile
          (4, 4, 5001, 128), (1, 3, 43, 128), (2, 2, 2500, 256), (2, 2, 300, 64), (1, 2, 200, 32)]


@pytest.mark.parametrize("io", ["f32", "bf16"])
@pytest.mark.parametrize("B,H,L,d", SHAPES)
def test_prepare_forward(io, B, H, L, d):
    x, s, _, got = _run(B, H, L, d, io)
    tol = 1e-5 if io == "f32" else 2e-2
    assert util.rel_err(got["q"], O.silu_l2norm(x["q_raw"], GP["norm_eps"])) <= tol
    assert util.rel_err(got["k"], O.silu_l2norm(x["k_raw"], GP["norm_eps"])) <= tol
    eta, beta, gamma = O.gates(s["a_eta"], s["a_beta"], s["a_alpha"], GP["eta_base"], GP["tau"], GP["alpha_base"])
    for n, ref in (("eta", eta), ("beta", beta), ("gamma", gamma)):
        assert util.rel_err(got[n], ref) <= 1e-5, n
    if io == "f32":
        assert np.allclose(np.sqrt((got["q"].astype(np.float64) ** 2).sum(-1)), 1.0, atol=1e-5)


@pytest.mark.parametrize("io", ["f32", "bf16"])
@pytest.mark.parametrize("B,H,L,d", SHAPES)
def test_prepare_backward(io, B, H, L, d):
    x, s, g, got = _run(B, H, L, d, io, seed=1, backward=True)
    tol = 1e-4 if io == "f32" else 2e-2
    assert util.rel_err(got["dq_raw"], O.silu_l2norm_vjp(x["q_raw"], x["dq"], GP["norm_eps"])) <= tol
    assert util.rel_err(got["dk_raw"], O.silu_l2norm_vjp(x["k_raw"], x["dk"], GP["norm_eps"])) <= tol
    da, db, dc = O.gates_vjp(s["a_eta"], s["a_beta"], s["a_alpha"], GP["eta_base"], GP["tau"], GP["alpha_base"],
                             g["d_eta"], g["d_beta"], g["d_gamma"])
    for n, ref in (("da_eta", da), ("da_beta", db), ("da_alpha", dc)):
        assert util.rel_err(got[n], ref) <= 1e-4, n


def test_prepare_feeds_the_chunk_update_in_the_papers_gate_regime():
    """Prepared tokens and gates go straight into e2ttt_chunk_fwd: keys have unit norm, gates sit in the paper's
    ranges, and the layer output agrees with the oracle run on the oracle-prepared inputs."""
    B, H, L, d = 1, 2, 128, 128
    x, s, _, got = _run(B, H, L, d, "bf16", seed=5)
    assert (got["eta"] > 0).all() and (got["eta"] < GP["eta_base"]).all()
    assert (got["beta"] > 0.8).all() and (got["beta"] < 1).all()          # tau = 32 pushes beta towards 1
    assert (got["gamma"] > 1 - GP["eta_base"] * GP["alpha_base"]).all() and (got["gamma"] < 1).all()
    r = inputs.Recipe(B=B * H, H=1, L=L, d=d, h=512, C=64, kind=inputs.KIND_MLP, io="bf16", seed=9)
    base = inputs.generate(r)
    xin = dict(base, q=got["q"].reshape(B * H, L, d), k=got["k"].reshape(B * H, L, d),
               eta=got["eta"].reshape(B * H, L), beta=got["beta"].reshape(B * H, L), gamma=got["gamma"].reshape(B * H, L))
    ref = util.oracle_forward(xin, 64, inputs.KIND_MLP)
    out, _ = util.gpu_forward(xin, d=d, h=512, C=64, kind=inputs.KIND_MLP, io="bf16")
    assert util.rel_err(out["o"], ref["o"]) <= 2e-2


@pytest.mark.parametrize("L", [9, 4000])
def test_prepare_forward_in_place(L):
    """q and k may alias q_raw and k_raw (both code paths: the per-row kernel and the bulk-copy pipeline)."""
    B, H, d = 2, 2, 128
    rng = np.random.default_rng(7)
    x = {n: _bf16(rng.standard_normal((B, H, L, d)).astype(np.float32)) for n in ("q_raw", "k_raw")}
    s = {n: rng.standard_normal((B, H, L)).astype(np.float32) for n in ("a_eta", "a_beta", "a_alpha")}
    p = E.make_params(B, H, L, d, 4 * d, 1, inputs.KIND_MLP, E.E2TTT_BF16, 1e-5, E.E2TTT_IMPL_AUTO)
    gp = E.e2ttt_gate_params(GP["eta_base"], GP["tau"], GP["alpha_base"], GP["norm_eps"])
    dev = lambda a, t=torch.float32: torch.tensor(a, dtype=torch.float32).to(t).cuda().contiguous()
    qr, kr = dev(x["q_raw"], torch.bfloat16), dev(x["k_raw"], torch.bfloat16)
    ae, ab, aa = dev(s["a_eta"]), dev(s["a_beta"]), dev(s["a_alpha"])
    q, k = torch.empty_like(qr), torch.empty_like(kr)
    eta, beta, gamma = torch.empty_like(ae), torch.empty_like(ae), torch.empty_like(ae)
    E.e2ttt_prepare_fwd(p, gp, qr, kr, ae, ab, aa, q, k, eta, beta, gamma)
    E.e2ttt_prepare_fwd(p, gp, qr, kr, ae, ab, aa, qr, kr, eta, beta, gamma)   # in place
    torch.cuda.synchronize()
    assert torch.equal(q, qr) and torch.equal(k, kr)
