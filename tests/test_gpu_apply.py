"""e2ttt_apply (outputs of fixed fast weights, the decode path) against the fp64 oracle, against the chunk forward's
own outputs, and as a streaming decoder: apply per token + one chunk update every C tokens == the one-shot forward."""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2608_21308_b200 import binding as E
from paper_2608_21308_b200 import inputs
from tests import util

pytestmark = pytest.mark.gpu
MLP, SWIGLU = inputs.KIND_MLP, inputs.KIND_SWIGLU
TOL_F32, TOL_BF16 = 1e-4, 2e-2


def gpu_apply(q, W, *, d, h, kind, io):
    N, T, _ = q.shape
    p = E.make_params(N, 1, T, d, h, 1, kind, E.E2TTT_F32 if io == "f32" else E.E2TTT_BF16, 1e-5, E.E2TTT_IMPL_AUTO)
    iod = torch.float32 if io == "f32" else torch.bfloat16
    qd = torch.tensor(q, dtype=torch.float32).to(iod).cuda().view(N, 1, T, d).contiguous()
    Wd = [torch.tensor(w, dtype=torch.float32).cuda().unsqueeze(1).contiguous() for w in W]
    o = torch.empty_like(qd)
    E.e2ttt_apply(p, qd, Wd, o)
    torch.cuda.synchronize()
    return o.float().cpu().numpy().reshape(N, T, d)


def oracle_apply(q, W, kind):
    N, T, d = q.shape
    out = np.empty((N, T, d))
    for n in range(N):
        Wn = [w[n] for w in W]
        for t in range(T):
            out[n, t] = oracle.net(Wn, q[n, t], kind)
    return out


@pytest.mark.parametrize("kind", [MLP, SWIGLU])
@pytest.mark.parametrize("io", ["f32", "bf16"])
@pytest.mark.parametrize("d,h,T,N", [(64, 256, 1, 2), (128, 512, 1, 3), (128, 384, 6, 2), (48, 80, 5, 3), (8, 16, 1, 1),
                                     (72, 136, 9, 2), (30, 50, 3, 2), (256, 1000, 2, 40)])
def test_apply_matches_oracle_net(kind, io, d, h, T, N):
    r = inputs.Recipe(B=N, H=1, L=T, d=d, h=h, C=max(T, 1), kind=kind, io=io, seed=21, w_std=0.05)
    x = inputs.generate(r)
    got = gpu_apply(x["q"], x["W"], d=d, h=h, kind=kind, io=io)
    ref = oracle_apply(x["q"], x["W"], kind)
    assert util.rel_err(got, ref) <= (TOL_F32 if io == "f32" else TOL_BF16)
    if io == "f32":
        assert util.rel_err(got, ref) <= 2e-6      # fp32 arithmetic on exact inputs: far inside the gate


def test_apply_equals_the_chunk_forwards_outputs_of_the_first_chunk():
    r = inputs.config(0, heads=[0, 1, 2])
    x = inputs.generate(r)
    fwd, _ = util.gpu_forward(x, d=r.d, h=r.h, C=r.C, kind=r.kind, io="f32")
    got = gpu_apply(x["q"][:, :r.C], x["W"], d=r.d, h=r.h, kind=r.kind, io="f32")
    assert util.rel_err(got, fwd["o"][:, :r.C]) <= 1e-5


@pytest.mark.parametrize("kind", [MLP, SWIGLU])
def test_streaming_decode_equals_one_shot_forward(kind):
    """Token by token: o_t from the chunk-start weights; after every C tokens the chunk update runs on the tokens
    that accumulated.  Outputs and the final state must equal the one-shot call (fp32 I/O, paper-regime gates)."""
    r = inputs.paper_regime(inputs.Recipe(B=2, H=1, L=64, d=32, h=64, C=16, kind=kind, io="f32", seed=5, m_std=0.002))
    x = inputs.generate(r)
    ref = util.oracle_forward(x, r.C, kind)
    shape = dict(d=r.d, h=r.h, C=r.C, kind=kind, io="f32")
    W, M = [w.copy() for w in x["W"]], [m.copy() for m in x["M"]]
    outs = []
    for t in range(r.L):
        outs.append(gpu_apply(x["q"][:, t:t + 1], W, d=r.d, h=r.h, kind=kind, io="f32"))
        if (t + 1) % r.C == 0:
            sl = slice(t + 1 - r.C, t + 1)
            chunk = {n: np.ascontiguousarray(x[n][:, sl]) for n in ("q", "k", "v", "eta", "beta", "gamma")}
            chunk["W"], chunk["M"] = W, M
            got, _ = util.gpu_forward(chunk, **shape)
            assert util.rel_err(got["o"], np.concatenate(outs[-r.C:], 1)) <= 1e-5   # the chunk call repeats those outputs
            W, M = got["W"], got["M"]
    o = np.concatenate(outs, 1)
    assert util.rel_err(o, ref["o"]) <= TOL_F32
    for i in range(len(W)):
        assert util.rel_err(W[i], ref["W"][i]) <= TOL_F32 and util.rel_err(M[i], ref["M"][i]) <= TOL_F32


def test_apply_at_the_benchmark_shape_sampled_against_the_oracle():
    r = inputs.config(2, L=1)
    x = inputs.generate(r)
    got = gpu_apply(x["q"], x["W"], d=r.d, h=r.h, kind=r.kind, io="bf16")
    heads = [0, 13, 31, 63]
    ref = oracle_apply(x["q"][heads], [w[heads] for w in x["W"]], r.kind)
    assert util.rel_err(got[heads], ref) <= TOL_BF16
    again = gpu_apply(x["q"], x["W"], d=r.d, h=r.h, kind=r.kind, io="bf16")
    assert np.array_equal(got, again)


def test_apply_rejects_bad_arguments():
    p = E.make_params(1, 1, 1, 64, 256, 1, MLP, E.E2TTT_F32, 1e-5, E.E2TTT_IMPL_AUTO)
    q = torch.zeros(1, 1, 1, 64, device="cuda")
    W = [torch.zeros(1, 1, 256, 64, device="cuda"), torch.zeros(1, 1, 64, 256, device="cuda")]
    with pytest.raises(Exception):
        E.e2ttt_apply(p, None, W, q)
    with pytest.raises(Exception):
        E.e2ttt_apply(p, q, W[:1], q)
