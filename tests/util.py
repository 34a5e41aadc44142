"""Helpers shared by the GPU parity tests: run the C-ABI library on numpy inputs, compare with the oracle."""
from __future__ import annotations

import numpy as np
import torch

from oracle import oracle
from paper_2608_21308_b200 import binding as E
from paper_2608_21308_b200 import inputs


def rel_err(x, ref) -> float:
    """max|x - ref| / max|ref| over one tensor (the gated parity metric)."""
    x = np.asarray(x, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    return float(np.max(np.abs(x - ref)) / max(float(np.max(np.abs(ref))), 1e-300))


def rel_l2(x, ref) -> float:
    x = np.asarray(x, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    return float(np.linalg.norm(x - ref) / max(float(np.linalg.norm(ref)), 1e-300))


def _dev(a, dtype):
    return torch.tensor(np.ascontiguousarray(a), dtype=torch.float32).to(dtype).cuda().contiguous()


def _io_dtype(io):
    return torch.float32 if io == "f32" else torch.bfloat16


def gpu_forward(x, *, d, h, C, kind, io, impl=E.E2TTT_IMPL_AUTO, eps=1e-5, save_states=False, use_M=True, ckpt_every=0):
    """x: dict from inputs.generate (arrays [N, ...]).  Runs e2ttt_chunk_fwd with B=N, H=1.  Returns numpy + handles."""
    N, L, _ = x["q"].shape
    p = E.make_params(N, 1, L, d, h, C, kind, E.E2TTT_F32 if io == "f32" else E.E2TTT_BF16, eps, impl, ckpt_every)
    iod = _io_dtype(io)
    q, k, v = (_dev(x[n], iod).view(N, 1, L, d) for n in ("q", "k", "v"))
    eta, beta, gamma = (_dev(x[n], torch.float32).view(N, 1, L) for n in ("eta", "beta", "gamma"))
    W = [_dev(w, torch.float32).unsqueeze(1).contiguous() for w in x["W"]]
    M = [_dev(m, torch.float32).unsqueeze(1).contiguous() for m in x["M"]] if use_M else None
    o = torch.empty_like(q)
    Wf = [torch.empty_like(w) for w in W]
    Mf = [torch.empty_like(w) for w in W]
    ws = torch.empty(E.e2ttt_workspace_bytes(p, int(save_states)), dtype=torch.uint8, device="cuda")
    E.e2ttt_chunk_fwd(p, q, k, v, eta, beta, gamma, W, M, o, Wf, Mf, ws, int(save_states))
    torch.cuda.synchronize()
    out = {"o": o.float().cpu().numpy().reshape(N, L, d),
           "W": [w.cpu().numpy()[:, 0] for w in Wf], "M": [m.cpu().numpy()[:, 0] for m in Mf]}
    handles = dict(p=p, q=q, k=k, v=v, eta=eta, beta=beta, gamma=gamma, W=W, M=M, ws=ws)
    return out, handles


def gpu_backward(x, *, d, h, C, kind, io, impl=E.E2TTT_IMPL_AUTO, eps=1e-5, use_M=True, use_dstate=True,
                 via_saved_states=False, ckpt_every=0, fwd_impl=None):
    N, L, _ = x["q"].shape
    p = E.make_params(N, 1, L, d, h, C, kind, E.E2TTT_F32 if io == "f32" else E.E2TTT_BF16, eps, impl, ckpt_every)
    iod = _io_dtype(io)
    q, k, v, d_o = (_dev(x[n], iod).view(N, 1, L, d) for n in ("q", "k", "v", "d_o"))
    eta, beta, gamma = (_dev(x[n], torch.float32).view(N, 1, L) for n in ("eta", "beta", "gamma"))
    W = [_dev(w, torch.float32).unsqueeze(1).contiguous() for w in x["W"]]
    M = [_dev(m, torch.float32).unsqueeze(1).contiguous() for m in x["M"]] if use_M else None
    dWf = [_dev(w, torch.float32).unsqueeze(1).contiguous() for w in x["dW"]] if use_dstate else None
    dMf = [_dev(w, torch.float32).unsqueeze(1).contiguous() for w in x["dM"]] if use_dstate else None
    dq, dk, dv = torch.empty_like(q), torch.empty_like(q), torch.empty_like(q)
    de, db, dg = torch.empty_like(eta), torch.empty_like(eta), torch.empty_like(eta)
    dW = [torch.empty_like(w) for w in W]
    dM = [torch.empty_like(w) for w in W]
    ws = torch.empty(E.e2ttt_workspace_bytes(p, 1), dtype=torch.uint8, device="cuda")
    if via_saved_states:
        o = torch.empty_like(q)
        Wf = [torch.empty_like(w) for w in W]
        Mf = [torch.empty_like(w) for w in W]
        pf = p
        if fwd_impl is not None:  # the forward on another kernel family than the backward (same workspace layout)
            pf = E.make_params(N, 1, L, d, h, C, kind, p.io_dtype, eps, fwd_impl, ckpt_every)
            assert E.e2ttt_workspace_bytes(pf, 1) == ws.numel()
        E.e2ttt_chunk_fwd(pf, q, k, v, eta, beta, gamma, W, M, o, Wf, Mf, ws, 1)
    E.e2ttt_chunk_bwd(p, q, k, v, eta, beta, gamma, W, M, d_o, dWf, dMf, dq, dk, dv, de, db, dg, dW, dM, ws,
                      int(via_saved_states))
    torch.cuda.synchronize()
    f = lambda t: t.float().cpu().numpy()
    return {"dq": f(dq).reshape(N, L, d), "dk": f(dk).reshape(N, L, d), "dv": f(dv).reshape(N, L, d),
            "deta": f(de).reshape(N, L), "dbeta": f(db).reshape(N, L), "dgamma": f(dg).reshape(N, L),
            "dW": [f(w)[:, 0] for w in dW], "dM": [f(m)[:, 0] for m in dM]}


def oracle_forward(x, C, kind, eps=1e-5, want_states=False, use_M=True):
    return oracle.forward(x["q"], x["k"], x["v"], x["eta"], x["beta"], x["gamma"], x["W"],
                          x["M"] if use_M else None, C, kind, eps=eps, want_states=want_states)


def oracle_backward(x, C, kind, eps=1e-5, use_M=True, use_dstate=True):
    return oracle.backward(x["q"], x["k"], x["v"], x["eta"], x["beta"], x["gamma"], x["W"],
                           x["M"] if use_M else None, x["d_o"], x["dW"] if use_dstate else None,
                           x["dM"] if use_dstate else None, C, kind, eps=eps)


def teacher_forced_windows(r: inputs.Recipe, n_chunks: int, window: int = 1, with_grads: bool = False):
    """Windows of `window` chunks, each started from the ORACLE's state at its first chunk.

    Runs the oracle over the first n_chunks chunks of the heads in r.heads, then returns (xw, ref):
      xw  - inputs of a batch whose "sequences" are the windows (N = heads * n_windows, L = window * C),
            W/M = the oracle's fp64 chunk-start states rounded to fp32 (what the library can be given);
      ref - the oracle re-run on exactly those fp32-rounded window inputs (so both sides start equal).
    """
    C = r.C
    rr = inputs.Recipe(**{**r.__dict__, "L": n_chunks * C})
    x = inputs.generate(rr, with_d_o=with_grads, with_dstate=False)
    full = oracle_forward(x, C, r.kind, want_states=True)
    N = x["q"].shape[0]
    nwin = n_chunks // window
    Lw = window * C
    shapes = inputs.mat_shapes(r.kind, r.d, r.h)
    nm = len(shapes)

    def cut(a):  # [N, n_chunks*C, ...] -> [N*nwin, Lw, ...]
        return np.ascontiguousarray(a[:, :nwin * Lw].reshape((N * nwin, Lw) + a.shape[2:]))

    xw = {n: cut(x[n]) for n in ("q", "k", "v", "eta", "beta", "gamma")}
    if with_grads:
        xw["d_o"] = cut(x["d_o"])
    st = full["states"][:, 0:nwin * window:window]  # [N, nwin, 2, nm, d*h]
    xw["W"] = [st[:, :, 0, i].reshape((N * nwin,) + shapes[i]).astype(np.float32) for i in range(nm)]
    xw["M"] = [st[:, :, 1, i].reshape((N * nwin,) + shapes[i]).astype(np.float32) for i in range(nm)]
    if with_grads:
        rng = np.random.Generator(np.random.Philox(key=[r.seed, 777]))
        xw["dW"] = [rng.standard_normal(w.shape).astype(np.float32) for w in xw["W"]]
        xw["dM"] = [rng.standard_normal(w.shape).astype(np.float32) for w in xw["W"]]
    ref = oracle_forward(xw, C, r.kind)
    return xw, ref


def teacher_forced_windows_at(r: inputs.Recipe, chunks, with_grads: bool = False):
    """One-chunk windows at the given chunk indices of a long sequence, each started from the ORACLE's state there.

    The oracle runs the sequence once from token 0 to the last requested chunk, in segments chained through its final
    state (a long run and the same run cut into calls are the same program), so no per-chunk states are stored.
    Returns (xw, ref) like teacher_forced_windows: N = heads * len(chunks) windows of L = C tokens.
    """
    C = r.C
    chunks = sorted(chunks)
    rr = inputs.Recipe(**{**r.__dict__, "L": (chunks[-1] + 1) * C})
    x = inputs.generate(rr, with_d_o=with_grads, with_dstate=False)
    N = x["q"].shape[0]
    shapes = inputs.mat_shapes(r.kind, r.d, r.h)
    nm = len(shapes)
    W = [w.astype(np.float64) for w in x["W"]]
    M = [m.astype(np.float64) for m in x["M"]]
    pos = 0
    starts = []
    for c in chunks:
        if c * C > pos:
            seg = {n: np.ascontiguousarray(x[n][:, pos:c * C]) for n in ("q", "k", "v", "eta", "beta", "gamma")}
            res = oracle.forward(seg["q"], seg["k"], seg["v"], seg["eta"], seg["beta"], seg["gamma"], W, M, C, r.kind)
            W, M = res["W"], res["M"]
            pos = c * C
        starts.append(([w.copy() for w in W], [m.copy() for m in M]))
    names = ("q", "k", "v", "eta", "beta", "gamma") + (("d_o",) if with_grads else ())
    xw = {n: np.ascontiguousarray(np.stack([x[n][:, c * C:(c + 1) * C] for c in chunks], axis=1).reshape((N * len(chunks), C) + x[n].shape[2:]))
          for n in names}
    xw["W"] = [np.stack([s[0][i] for s in starts], axis=1).reshape((N * len(chunks),) + shapes[i]).astype(np.float32) for i in range(nm)]
    xw["M"] = [np.stack([s[1][i] for s in starts], axis=1).reshape((N * len(chunks),) + shapes[i]).astype(np.float32) for i in range(nm)]
    if with_grads:
        rng = np.random.Generator(np.random.Philox(key=[r.seed, 778]))
        xw["dW"] = [rng.standard_normal(w.shape).astype(np.float32) for w in xw["W"]]
        xw["dM"] = [rng.standard_normal(w.shape).astype(np.float32) for w in xw["W"]]
    ref = oracle_forward(xw, C, r.kind)
    return xw, ref
