"""Seeded synthetic inputs for the E2-TTT chunk update.

This module is data only: it draws the tensors a call consumes and rounds them to the
I/O dtype.  It holds none of the method's arithmetic (no scans, no fast-weight network,
no state update) so that the CPU oracle and the CUDA path can both be fed from it
without sharing any code of their own.

Every tensor of every (batch, head) pair comes from its own counter-based Philox
stream keyed by (seed, tensor id, b*H + h), so one head can be generated alone and is
identical to the same head inside a full batch.

Distributions (the benchmark recipe; the paper's own gate regime is the "paper"
variant, Table "Model hyperparameters" and the equations for eta, beta and gamma in the
section "Input-Dependent Dynamics"):

  q, v      i.i.d. N(0, 1)
  k         i.i.d. N(0, 1), then every token vector scaled to unit L2 norm
  eta       eta_base * sigmoid(N(0, 1))
  beta      sigmoid(N(1, 1)) ** (1 / tau)
  alpha     alpha_base * sigmoid(N(3, 1))
  gamma     gates == "coupled": 1 - eta * alpha   (decoupled weight-decay form)
            gates == "direct" : alpha             (alpha read as the forget gate itself)
  W_init    every fast-weight matrix i.i.d. N(0, w_std)
  M_init    zeros, or N(0, m_std) when m_std > 0
  d_o       i.i.d. N(0, 1)
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

KIND_MLP = 0
KIND_SWIGLU = 1

_TENSOR_IDS = {"q": 1, "k": 2, "v": 3, "eta": 4, "beta": 5, "alpha": 6, "W": 7, "M": 8, "d_o": 9,
               "dW": 10, "dM": 11}


def mat_shapes(kind: int, d: int, h: int):
    """Row-major shapes of the fast-weight matrices: MLP (W1[h,d], W2[d,h]); SwiGLU (W1[h,d], W2[h,d], W3[d,h])."""
    if kind == KIND_MLP:
        return [(h, d), (d, h)]
    if kind == KIND_SWIGLU:
        return [(h, d), (h, d), (d, h)]
    raise ValueError(f"unknown kind {kind}")


def swiglu_hidden(d: int) -> int:
    """(8/3) d rounded up to a multiple of 64 (384 at d=128, 192 at d=64)."""
    return 64 * ((8 * d + 3 * 64 - 1) // (3 * 64))


def round_bf16(x: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bf16 (ties to even); returns fp32 holding bf16-representable values."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    bias = ((u >> 16) & 1) + np.uint32(0x7FFF)
    r = ((u + bias) & np.uint32(0xFFFF0000)).astype(np.uint32)
    return r.view(np.float32)


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32 array whose values are already bf16-representable -> uint16 bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    return (x.view(np.uint32) >> 16).astype(np.uint16)


def from_bf16_bits(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << 16).view(np.float32)


@dataclass
class Recipe:
    B: int
    H: int
    L: int
    d: int
    h: int
    C: int
    kind: int = KIND_MLP
    io: str = "f32"            # "f32" | "bf16": dtype q, k, v (and d_o) are rounded to
    seed: int = 0
    gates: str = "coupled"     # "coupled" | "direct"
    eta_base: float = 0.1
    tau: float = 1.0
    alpha_base: float = 1.0
    w_std: float = 0.02
    m_std: float = 0.0
    heads: list | None = None  # subset of flat head indices b*H+h to generate (None = all)
    extra: dict = field(default_factory=dict)


def paper_regime(r: Recipe) -> Recipe:
    """Same shapes, the paper's gate bases: eta_base 0.01, tau 32, alpha_base 0.1."""
    return Recipe(**{**r.__dict__, "eta_base": 0.01, "tau": 32.0, "alpha_base": 0.1, "gates": "coupled"})


def _rng(seed: int, name: str, head: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[(seed << 8) | _TENSOR_IDS[name], head]))


def _sigmoid(x):
    return 1.0 / (1.0 + np.exp(-x))


def generate(r: Recipe, with_d_o: bool = False, with_dstate: bool = False) -> dict:
    """Draw one call's inputs.

    Returns fp32 numpy arrays: q, k, v [N, L, d]; eta, beta, gamma [N, L]; W (list of
    [N, rows, cols]); M (same, zeros unless m_std > 0); optionally d_o [N, L, d] and
    dW / dM (N(0,1) adjoints of the final state).  N = B*H, or len(r.heads).
    q, k, v and d_o hold values already rounded to r.io.
    """
    heads = list(range(r.B * r.H)) if r.heads is None else list(r.heads)
    N, L, d = len(heads), r.L, r.d
    shapes = mat_shapes(r.kind, r.d, r.h)
    out = {
        "q": np.empty((N, L, d), np.float32), "k": np.empty((N, L, d), np.float32),
        "v": np.empty((N, L, d), np.float32),
        "eta": np.empty((N, L), np.float32), "beta": np.empty((N, L), np.float32),
        "gamma": np.empty((N, L), np.float32),
        "W": [np.empty((N,) + s, np.float32) for s in shapes],
        "M": [np.zeros((N,) + s, np.float32) for s in shapes],
    }
    if with_d_o:
        out["d_o"] = np.empty((N, L, d), np.float32)
    if with_dstate:
        out["dW"] = [np.empty((N,) + s, np.float32) for s in shapes]
        out["dM"] = [np.empty((N,) + s, np.float32) for s in shapes]
    for n, head in enumerate(heads):
        out["q"][n] = _rng(r.seed, "q", head).standard_normal((L, d), dtype=np.float32)
        kk = _rng(r.seed, "k", head).standard_normal((L, d), dtype=np.float32)
        kk /= np.sqrt((kk.astype(np.float64) ** 2).sum(-1, keepdims=True)).astype(np.float32)
        out["k"][n] = kk
        out["v"][n] = _rng(r.seed, "v", head).standard_normal((L, d), dtype=np.float32)
        eta = r.eta_base * _sigmoid(_rng(r.seed, "eta", head).standard_normal(L))
        beta = _sigmoid(1.0 + _rng(r.seed, "beta", head).standard_normal(L)) ** (1.0 / r.tau)
        alpha = r.alpha_base * _sigmoid(3.0 + _rng(r.seed, "alpha", head).standard_normal(L))
        gamma = 1.0 - eta * alpha if r.gates == "coupled" else alpha
        out["eta"][n], out["beta"][n], out["gamma"][n] = eta, beta, gamma
        gw = _rng(r.seed, "W", head)
        gm = _rng(r.seed, "M", head)
        for i, s in enumerate(shapes):
            out["W"][i][n] = r.w_std * gw.standard_normal(s, dtype=np.float32)
            if r.m_std > 0:
                out["M"][i][n] = r.m_std * gm.standard_normal(s, dtype=np.float32)
        if with_d_o:
            out["d_o"][n] = _rng(r.seed, "d_o", head).standard_normal((L, d), dtype=np.float32)
        if with_dstate:
            gdw, gdm = _rng(r.seed, "dW", head), _rng(r.seed, "dM", head)
            for i, s in enumerate(shapes):
                out["dW"][i][n] = gdw.standard_normal(s, dtype=np.float32)
                out["dM"][i][n] = gdm.standard_normal(s, dtype=np.float32)
    if r.io == "bf16":
        for name in ("q", "k", "v") + (("d_o",) if with_d_o else ()):
            out[name] = round_bf16(out[name])
    elif r.io != "f32":
        raise ValueError(f"unknown io dtype {r.io}")
    return out


# The five benchmark configurations (shapes and distributions as the benchmark states them).
def config(i: int, **over) -> Recipe:
    base = [
        dict(B=1, H=1, L=256, d=64, h=256, C=16, kind=KIND_MLP, io="f32"),
        dict(B=8, H=12, L=2048, d=64, h=256, C=64, kind=KIND_MLP, io="bf16"),
        dict(B=4, H=16, L=4096, d=128, h=512, C=64, kind=KIND_MLP, io="bf16"),
        dict(B=4, H=16, L=4096, d=128, h=swiglu_hidden(128), C=64, kind=KIND_SWIGLU, io="bf16"),
        dict(B=1, H=16, L=32768, d=128, h=512, C=64, kind=KIND_MLP, io="bf16"),
    ][i]
    base.update(over)
    return Recipe(**base)
