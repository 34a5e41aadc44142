"""ctypes front end of the fp64 CPU oracle (oracle/e2ttt_oracle.c).

TEST INFRASTRUCTURE ONLY.  Imported by tests/, by the smoke check and by the benchmark's
CPU-baseline leg; never by the CUDA package.  Imports nothing from that package either.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import sys

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "e2ttt_oracle.c")
_LIB = os.path.join(_HERE, "build", "libe2ttt_oracle.so")

KIND_MLP = 0
KIND_SWIGLU = 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP over independent sequences only)."""
    if not force and os.path.exists(_LIB) and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC):
        return _LIB
    os.makedirs(os.path.dirname(_LIB), exist_ok=True)
    tmp = _LIB + f".tmp{os.getpid()}"
    cmd = ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.e2ttt_oracle_inner.restype = ctypes.c_double
    return _lib


def nmat(kind: int) -> int:
    return 2 if kind == KIND_MLP else 3


def mat_shapes(kind: int, d: int, h: int):
    return [(h, d), (d, h)] if kind == KIND_MLP else [(h, d), (h, d), (d, h)]


_dp = ctypes.POINTER(ctypes.c_double)


def _p(a):
    return None if a is None else a.ctypes.data_as(_dp)


def _pp(lst):
    if lst is None:
        return None
    arr = (_dp * len(lst))(*[_p(a) for a in lst])
    return arr


def _f64(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float64)


def _f64l(lst):
    return None if lst is None else [_f64(a) for a in lst]


def forward(q, k, v, eta, beta, gamma, W_init, M_init, C, kind, eps=1e-5, threads=0, want_states=False,
            row_norm=None, norm_eps=1e-5):
    """q, k, v [N, L, d]; gates [N, L]; W_init list of [N, rows, cols]; M_init same or None.

    row_norm: None, or a list of [N, rows_i] target norms: every row of every W_i is rescaled to its target after
    each chunk (post-chunk normalisation).
    Returns dict(o, W, M[, states]) in fp64; states [N, nchunks, 2, nmat, d*h] holds (W, M) at chunk starts.
    """
    q, k, v, eta, beta, gamma = map(_f64, (q, k, v, eta, beta, gamma))
    W_init, M_init = _f64l(W_init), _f64l(M_init)
    N, L, d = q.shape
    h = W_init[0].shape[1]
    shapes = mat_shapes(kind, d, h)
    assert [w.shape[1:] for w in W_init] == shapes, "fast-weight shapes do not match kind/d/h"
    o = np.empty((N, L, d))
    Wf = [np.empty((N,) + s) for s in shapes]
    Mf = [np.empty((N,) + s) for s in shapes]
    nchunks = (L + C - 1) // C
    states = np.empty((N, nchunks, 2, len(shapes), d * h)) if want_states else None
    row_norm = _f64l(row_norm)
    rc = lib().e2ttt_oracle_fwd_norm(
        N, L, d, h, C, kind, ctypes.c_double(eps), _p(q), _p(k), _p(v), _p(eta), _p(beta), _p(gamma),
        _pp(W_init), _pp(M_init), _p(o), _pp(Wf), _pp(Mf), _p(states), threads, _pp(row_norm),
        ctypes.c_double(norm_eps))
    if rc != 0:
        raise RuntimeError("oracle forward failed")
    out = {"o": o, "W": Wf, "M": Mf}
    if want_states:
        out["states"] = states
    return out


def backward(q, k, v, eta, beta, gamma, W_init, M_init, d_o, dW_final, dM_final, C, kind, eps=1e-5, threads=0,
             row_norm=None, norm_eps=1e-5):
    """Adjoints of every input of forward(), given d_o and (optional) adjoints of the final state.
    With row_norm the result also holds "drow_norm", the adjoints of the target norms."""
    q, k, v, eta, beta, gamma, d_o = map(_f64, (q, k, v, eta, beta, gamma, d_o))
    W_init, M_init, dW_final, dM_final = map(_f64l, (W_init, M_init, dW_final, dM_final))
    N, L, d = q.shape
    h = W_init[0].shape[1]
    shapes = mat_shapes(kind, d, h)
    dq, dk, dv = np.empty((N, L, d)), np.empty((N, L, d)), np.empty((N, L, d))
    de, db, dg = np.empty((N, L)), np.empty((N, L)), np.empty((N, L))
    dW = [np.empty((N,) + s) for s in shapes]
    dM = [np.empty((N,) + s) for s in shapes]
    row_norm = _f64l(row_norm)
    drn = [np.zeros((N, s[0])) for s in shapes] if row_norm is not None else None
    rc = lib().e2ttt_oracle_bwd_norm(
        N, L, d, h, C, kind, ctypes.c_double(eps), _p(q), _p(k), _p(v), _p(eta), _p(beta), _p(gamma),
        _pp(W_init), _pp(M_init), _p(d_o), _pp(dW_final), _pp(dM_final),
        _p(dq), _p(dk), _p(dv), _p(de), _p(db), _p(dg), _pp(dW), _pp(dM), threads, _pp(row_norm),
        ctypes.c_double(norm_eps), _pp(drn))
    if rc != 0:
        raise RuntimeError("oracle backward failed")
    out = {"dq": dq, "dk": dk, "dv": dv, "deta": de, "dbeta": db, "dgamma": dg, "dW": dW, "dM": dM}
    if drn is not None:
        out["drow_norm"] = drn
    return out


def inner(W, k, v, kind, eps=1e-5, want_grad=True):
    """One token at fixed weights W (list of [rows, cols]): returns (loss, G list or None), G = -dL/dW."""
    W = _f64l(W)
    k, v = _f64(k), _f64(v)
    d = k.shape[0]
    h = W[0].shape[0]
    G = [np.empty_like(w) for w in W] if want_grad else None
    loss = lib().e2ttt_oracle_inner(d, h, kind, ctypes.c_double(eps), _pp(W), _p(k), _p(v), _pp(G))
    return float(loss), G


def net(W, x, kind, eps=1e-5):
    """f_W(x) for one token."""
    W = _f64l(W)
    x = _f64(x)
    d = x.shape[0]
    h = W[0].shape[0]
    out = np.empty(d)
    rc = lib().e2ttt_oracle_net(d, h, kind, ctypes.c_double(eps), _pp(W), _p(x), _p(out))
    if rc != 0:
        raise RuntimeError("oracle net failed")
    return out


def max_threads() -> int:
    return int(lib().e2ttt_oracle_max_threads())


if __name__ == "__main__":
    print(build(force="--force" in sys.argv))
