"""The calls only enqueue work on the caller's stream: they run on a side stream, and they can be captured in a CUDA
graph and replayed (nothing is allocated, the host is never synchronised)."""
import numpy as np
import pytest
import torch

from paper_2608_21308_b200 import binding as E
from paper_2608_21308_b200 import inputs

pytestmark = pytest.mark.gpu


def _setup(r, impl):
    x = inputs.generate(r)
    N, L, d = x["q"].shape
    p = E.make_params(N, 1, L, d, r.h, r.C, r.kind, E.E2TTT_BF16, 1e-5, impl)
    dev = lambda a, t=torch.float32: torch.tensor(a, dtype=torch.float32).to(t).cuda().contiguous()
    q, k, v = (dev(x[n], torch.bfloat16).view(N, 1, L, d) for n in ("q", "k", "v"))
    eta, beta, gamma = (dev(x[n]).view(N, 1, L) for n in ("eta", "beta", "gamma"))
    W = [dev(w).unsqueeze(1).contiguous() for w in x["W"]]
    o = torch.zeros_like(q)
    Wf = [torch.zeros_like(w) for w in W]
    Mf = [torch.zeros_like(w) for w in W]
    ws = torch.empty(E.e2ttt_workspace_bytes(p, 0), dtype=torch.uint8, device="cuda")
    return p, (q, k, v, eta, beta, gamma, W), (o, Wf, Mf), ws


@pytest.mark.parametrize("cfg,impl", [(2, E.E2TTT_IMPL_TCGEN05), (3, E.E2TTT_IMPL_TILED)], ids=["fused", "tiled"])
def test_forward_on_a_side_stream_and_from_a_cuda_graph(cfg, impl):
    r = inputs.config(cfg, heads=[0, 1, 2], L=256)
    p, (q, k, v, eta, beta, gamma, W), (o, Wf, Mf), ws = _setup(r, impl)
    E.e2ttt_chunk_fwd(p, q, k, v, eta, beta, gamma, W, None, o, Wf, Mf, ws, 0)          # eager, default stream
    torch.cuda.synchronize()
    ref = (o.clone(), [w.clone() for w in Wf], [m.clone() for m in Mf])

    side = torch.cuda.Stream()
    for t in (o, *Wf, *Mf):
        t.zero_()
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        E.e2ttt_chunk_fwd(p, q, k, v, eta, beta, gamma, W, None, o, Wf, Mf, ws, 0, side)
    side.synchronize()
    assert torch.equal(o, ref[0]) and all(torch.equal(a, b) for a, b in zip(Wf + Mf, ref[1] + ref[2]))

    for t in (o, *Wf, *Mf):
        t.zero_()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        E.e2ttt_chunk_fwd(p, q, k, v, eta, beta, gamma, W, None, o, Wf, Mf, ws, 0, torch.cuda.current_stream())
    for t in (o, *Wf, *Mf):
        t.zero_()
    graph.replay()
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(o, ref[0]) and all(torch.equal(a, b) for a, b in zip(Wf + Mf, ref[1] + ref[2]))
    assert E.e2ttt_device_status(ws) == 0


def test_decode_loop_from_a_cuda_graph():
    """One graph = C applies (one token each) followed by the chunk update: replayed for the next chunk it continues."""
    r = inputs.paper_regime(inputs.Recipe(B=2, H=1, L=128, d=128, h=512, C=64, kind=inputs.KIND_MLP, io="bf16", seed=3))
    p, (q, k, v, eta, beta, gamma, W), (o, Wf, Mf), ws = _setup(r, E.E2TTT_IMPL_AUTO)
    E.e2ttt_chunk_fwd(p, q, k, v, eta, beta, gamma, W, None, o, Wf, Mf, ws, 0)
    torch.cuda.synchronize()
    ref_o = o.clone()
    N, C, d = 2, 64, 128
    p1 = E.make_params(N, 1, 1, d, 512, 1, inputs.KIND_MLP, E.E2TTT_BF16, 1e-5, E.E2TTT_IMPL_AUTO)
    pc = E.make_params(N, 1, C, d, 512, C, inputs.KIND_MLP, E.E2TTT_BF16, 1e-5, E.E2TTT_IMPL_AUTO)
    # static buffers the graph works on: the chunk's tokens, the running state, the outputs
    cq, ck, cv = (torch.empty(N, 1, C, d, dtype=torch.bfloat16, device="cuda") for _ in range(3))
    ce, cb, cg = (torch.empty(N, 1, C, device="cuda") for _ in range(3))
    Wc = [w.clone() for w in W]
    Mc = [torch.zeros_like(w) for w in W]
    co = torch.empty_like(cq)
    tok_q = [torch.empty(N, 1, 1, d, dtype=torch.bfloat16, device="cuda") for _ in range(C)]
    tok_o = [torch.empty(N, 1, 1, d, dtype=torch.bfloat16, device="cuda") for _ in range(C)]
    wsc = torch.empty(E.e2ttt_workspace_bytes(pc, 0), dtype=torch.uint8, device="cuda")

    def body(stream):
        for t in range(C):
            E.e2ttt_apply(p1, tok_q[t], Wc, tok_o[t], stream)
        E.e2ttt_chunk_fwd(pc, cq, ck, cv, ce, cb, cg, Wc, Mc, co, Wc, Mc, wsc, 0, stream)   # in-place state update

    def load(c):
        sl = slice(c * C, (c + 1) * C)
        cq.copy_(q[:, :, sl]); ck.copy_(k[:, :, sl]); cv.copy_(v[:, :, sl])
        ce.copy_(eta[:, :, sl]); cb.copy_(beta[:, :, sl]); cg.copy_(gamma[:, :, sl])
        for t in range(C):
            tok_q[t].copy_(q[:, :, c * C + t:c * C + t + 1])

    load(0)
    body(torch.cuda.current_stream())      # warm-up outside the graph (first-call attribute setup)
    for w_dst, w_src in zip(Wc, W):
        w_dst.copy_(w_src)
    for m in Mc:
        m.zero_()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        body(torch.cuda.current_stream())
    for w_dst, w_src in zip(Wc, W):        # capture does not run the work; start from the initial state
        w_dst.copy_(w_src)
    for m in Mc:
        m.zero_()
    outs = []
    for c in range(r.L // C):
        load(c)
        graph.replay()
        torch.cuda.synchronize()
        outs.append(torch.cat([t.clone() for t in tok_o], 2))
        # the chunk call repeats the outputs of its tokens (fp32 apply vs bf16-operand chunk kernel: bf16-level agreement)
        a_, b_ = outs[-1].float(), co.float()
        assert float((a_ - b_).abs().max() / b_.abs().max()) <= 2e-2
    got = torch.cat(outs, 2).float().cpu().numpy()
    refn = ref_o.float().cpu().numpy()
    # apply computes in fp32 from the fp32 weights, the fused chunk kernel with bf16 operands: bf16-level agreement
    assert float(np.max(np.abs(got - refn)) / np.max(np.abs(refn))) <= 2e-2
