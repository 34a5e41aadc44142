"""Thin ctypes binding of the C-ABI library (include/e2ttt.h): argument marshalling only.

Every function has the name and the argument order of its C counterpart.  Tensors are torch CUDA
tensors (torch is used for device memory and streams, nothing else); the binding checks dtype,
contiguity and device, builds the host pointer tables and passes raw pointers.  There is no CPU
path: a missing library or a failing call raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "lib", "libe2ttt.so")

E2TTT_MLP_GELU, E2TTT_SWIGLU = 0, 1
E2TTT_F32, E2TTT_BF16 = 0, 1
E2TTT_IMPL_AUTO, E2TTT_IMPL_SIMT, E2TTT_IMPL_TCGEN05, E2TTT_IMPL_TILED = 0, 1, 2, 3
E2TTT_OK = 0


class e2ttt_gate_params(ctypes.Structure):
    _fields_ = [("eta_base", ctypes.c_float), ("tau", ctypes.c_float), ("alpha_base", ctypes.c_float),
                ("norm_eps", ctypes.c_float)]


class e2ttt_params(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("H", ctypes.c_int32), ("L", ctypes.c_int32), ("d", ctypes.c_int32),
                ("h", ctypes.c_int32), ("C", ctypes.c_int32), ("kind", ctypes.c_int32),
                ("io_dtype", ctypes.c_int32), ("ln_eps", ctypes.c_float), ("impl", ctypes.c_int32),
                ("ckpt_every", ctypes.c_int32)]


class E2TTTError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {e2ttt_status_string(status)} ({status})")


_lib = None


def lib() -> ctypes.CDLL:
    """Load the in-tree library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} not found: build it with `python -m paper_2608_21308_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        vp, cp = ctypes.c_void_p, ctypes.c_int
        pp = ctypes.POINTER(e2ttt_params)
        tab = ctypes.POINTER(ctypes.c_void_p)
        L.e2ttt_num_matrices.argtypes = [cp]
        L.e2ttt_matrix_shape.argtypes = [cp, cp, cp, cp, ctypes.POINTER(cp), ctypes.POINTER(cp)]
        L.e2ttt_workspace_bytes.argtypes = [pp, cp, ctypes.POINTER(ctypes.c_size_t)]
        L.e2ttt_workspace_bytes_normed.argtypes = [pp, cp, ctypes.POINTER(ctypes.c_size_t)]
        L.e2ttt_workspace_bytes_normed.restype = cp
        L.e2ttt_chunk_fwd.argtypes = [pp, vp, vp, vp, vp, vp, vp, tab, tab, vp, tab, tab, vp, ctypes.c_size_t, cp, vp]
        L.e2ttt_chunk_bwd.argtypes = [pp, vp, vp, vp, vp, vp, vp, tab, tab, vp, tab, tab, vp, vp, vp, vp, vp, vp,
                                      tab, tab, vp, ctypes.c_size_t, cp, vp]
        L.e2ttt_chunk_fwd_noalloc.argtypes = [pp, vp, vp, vp, vp, vp, vp, tab, tab, vp, tab, tab, vp]
        L.e2ttt_chunk_fwd_noalloc.restype = cp
        L.e2ttt_chunk_fwd_normed.argtypes = [pp, vp, vp, vp, vp, vp, vp, tab, tab, tab, ctypes.c_float, vp, tab, tab, vp,
                                             ctypes.c_size_t, cp, vp]
        L.e2ttt_chunk_fwd_normed.restype = cp
        L.e2ttt_chunk_bwd_normed.argtypes = [pp, vp, vp, vp, vp, vp, vp, tab, tab, tab, ctypes.c_float, vp, tab, tab, vp, vp,
                                             vp, vp, vp, vp, tab, tab, tab, vp, ctypes.c_size_t, cp, vp]
        L.e2ttt_chunk_bwd_normed.restype = cp
        gp = ctypes.POINTER(e2ttt_gate_params)
        L.e2ttt_prepare_fwd.argtypes = [pp, gp] + [vp] * 11
        L.e2ttt_prepare_fwd.restype = cp
        L.e2ttt_prepare_bwd.argtypes = [pp, gp] + [vp] * 16
        L.e2ttt_prepare_bwd.restype = cp
        L.e2ttt_apply.argtypes = [pp, vp, tab, vp, vp]
        L.e2ttt_apply.restype = cp
        L.e2ttt_device_status.argtypes = [vp, vp, ctypes.POINTER(cp)]
        L.e2ttt_device_status.restype = cp
        L.e2ttt_selftest_wait_timeout.argtypes = [vp, ctypes.c_size_t, ctypes.c_longlong, vp]
        L.e2ttt_selftest_wait_timeout.restype = cp
        L.e2ttt_status_string.argtypes = [cp]
        L.e2ttt_status_string.restype = ctypes.c_char_p
        L.e2ttt_version.argtypes = []
        for name in ("e2ttt_num_matrices", "e2ttt_matrix_shape", "e2ttt_workspace_bytes", "e2ttt_chunk_fwd",
                     "e2ttt_chunk_bwd", "e2ttt_version"):
            getattr(L, name).restype = cp
        _lib = L
    return _lib


def e2ttt_status_string(status: int) -> str:
    return lib().e2ttt_status_string(int(status)).decode()


def e2ttt_version() -> int:
    return int(lib().e2ttt_version())


def e2ttt_num_matrices(kind: int) -> int:
    return int(lib().e2ttt_num_matrices(int(kind)))


def e2ttt_matrix_shape(kind: int, d: int, h: int, i: int):
    r, c = ctypes.c_int(), ctypes.c_int()
    st = lib().e2ttt_matrix_shape(kind, d, h, i, ctypes.byref(r), ctypes.byref(c))
    if st != E2TTT_OK:
        raise E2TTTError(st, "e2ttt_matrix_shape")
    return r.value, c.value


def e2ttt_workspace_bytes(p: e2ttt_params, save_states: int) -> int:
    n = ctypes.c_size_t()
    st = lib().e2ttt_workspace_bytes(ctypes.byref(p), int(save_states), ctypes.byref(n))
    if st != E2TTT_OK:
        raise E2TTTError(st, "e2ttt_workspace_bytes")
    return int(n.value)


def e2ttt_workspace_bytes_normed(p: e2ttt_params, save_states: int) -> int:
    n = ctypes.c_size_t()
    st = lib().e2ttt_workspace_bytes_normed(ctypes.byref(p), int(save_states), ctypes.byref(n))
    if st != E2TTT_OK:
        raise E2TTTError(st, "e2ttt_workspace_bytes_normed")
    return int(n.value)


def make_params(B, H, L, d, h, C, kind=E2TTT_MLP_GELU, io_dtype=E2TTT_F32, ln_eps=1e-5, impl=E2TTT_IMPL_AUTO,
                ckpt_every=0):
    return e2ttt_params(B, H, L, d, h, C, kind, io_dtype, ln_eps, impl, ckpt_every)


def _io_torch_dtype(p):
    return torch.float32 if p.io_dtype == E2TTT_F32 else torch.bfloat16


def _ptr(t, dtype, shape, name):
    if t is None:
        return None
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError(f"{name}: expected a CUDA tensor")
    if t.dtype != dtype:
        raise TypeError(f"{name}: expected dtype {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{name}: must be contiguous")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name}: expected shape {tuple(shape)}, got {tuple(t.shape)}")
    return ctypes.c_void_p(t.data_ptr())


def _table(ts, p, name):
    if ts is None:
        return None
    n = e2ttt_num_matrices(p.kind)
    if len(ts) != n:
        raise ValueError(f"{name}: expected {n} matrices")
    arr = (ctypes.c_void_p * n)()
    for i, t in enumerate(ts):
        r, c = e2ttt_matrix_shape(p.kind, p.d, p.h, i)
        arr[i] = _ptr(t, torch.float32, (p.B, p.H, r, c), f"{name}[{i}]")
    return arr


def _stream_ptr(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream if isinstance(stream, torch.cuda.Stream) else int(stream))


def e2ttt_chunk_fwd(p, q, k, v, eta, beta, gamma, W_init, M_init, o, W_final, M_final, workspace,
                    save_states=0, stream=None):
    """int e2ttt_chunk_fwd(...) of include/e2ttt.h.  `workspace` is a uint8 CUDA tensor.  Raises on error."""
    io = _io_torch_dtype(p)
    s4, s3 = (p.B, p.H, p.L, p.d), (p.B, p.H, p.L)
    st = lib().e2ttt_chunk_fwd(
        ctypes.byref(p), _ptr(q, io, s4, "q"), _ptr(k, io, s4, "k"), _ptr(v, io, s4, "v"),
        _ptr(eta, torch.float32, s3, "eta"), _ptr(beta, torch.float32, s3, "beta"),
        _ptr(gamma, torch.float32, s3, "gamma"), _table(W_init, p, "W_init"), _table(M_init, p, "M_init"),
        _ptr(o, io, s4, "o"), _table(W_final, p, "W_final"), _table(M_final, p, "M_final"),
        _ptr(workspace, torch.uint8, None, "workspace"), workspace.numel() if workspace is not None else 0,
        int(save_states), _stream_ptr(stream))
    if st != E2TTT_OK:
        raise E2TTTError(st, "e2ttt_chunk_fwd")
    return st


def _row_table(ts, p, name):
    """nmat pointers to [B, H, rows_i] fp32 tensors (row targets of the post-chunk normalisation, or their adjoints)."""
    if ts is None:
        return None
    n = e2ttt_num_matrices(p.kind)
    if len(ts) != n:
        raise ValueError(f"{name}: expected {n} tensors")
    arr = (ctypes.c_void_p * n)()
    for i, t in enumerate(ts):
        r, _ = e2ttt_matrix_shape(p.kind, p.d, p.h, i)
        arr[i] = _ptr(t, torch.float32, (p.B, p.H, r), f"{name}[{i}]")
    return arr


def e2ttt_chunk_fwd_normed(p, q, k, v, eta, beta, gamma, W_init, M_init, row_norm, norm_eps, o, W_final, M_final,
                           workspace, save_states=0, stream=None):
    """int e2ttt_chunk_fwd_normed(...) of include/e2ttt.h.  Raises on error."""
    io = _io_torch_dtype(p)
    s4, s3 = (p.B, p.H, p.L, p.d), (p.B, p.H, p.L)
    st = lib().e2ttt_chunk_fwd_normed(
        ctypes.byref(p), _ptr(q, io, s4, "q"), _ptr(k, io, s4, "k"), _ptr(v, io, s4, "v"),
        _ptr(eta, torch.float32, s3, "eta"), _ptr(beta, torch.float32, s3, "beta"),
        _ptr(gamma, torch.float32, s3, "gamma"), _table(W_init, p, "W_init"), _table(M_init, p, "M_init"),
        _row_table(row_norm, p, "row_norm"), float(norm_eps),
        _ptr(o, io, s4, "o"), _table(W_final, p, "W_final"), _table(M_final, p, "M_final"),
        _ptr(workspace, torch.uint8, None, "workspace"), workspace.numel() if workspace is not None else 0,
        int(save_states), _stream_ptr(stream))
    if st != E2TTT_OK:
        raise E2TTTError(st, "e2ttt_chunk_fwd_normed")
    return st


def e2ttt_chunk_bwd_normed(p, q, k, v, eta, beta, gamma, W_init, M_init, row_norm, norm_eps, d_o, dW_final, dM_final,
                           dq, dk, dv, d_eta, d_beta, d_gamma, dW_init, dM_init, d_row_norm, workspace,
                           states_saved=0, stream=None):
    """int e2ttt_chunk_bwd_normed(...) of include/e2ttt.h.  Raises on error."""
    io = _io_torch_dtype(p)
    s4, s3 = (p.B, p.H, p.L, p.d), (p.B, p.H, p.L)
    f32 = torch.float32
    st = lib().e2ttt_chunk_bwd_normed(
        ctypes.byref(p), _ptr(q, io, s4, "q"), _ptr(k, io, s4, "k"), _ptr(v, io, s4, "v"),
        _ptr(eta, f32, s3, "eta"), _ptr(beta, f32, s3, "beta"), _ptr(gamma, f32, s3, "gamma"),
        _table(W_init, p, "W_init"), _table(M_init, p, "M_init"), _row_table(row_norm, p, "row_norm"), float(norm_eps),
        _ptr(d_o, io, s4, "d_o"), _table(dW_final, p, "dW_final"), _table(dM_final, p, "dM_final"),
        _ptr(dq, io, s4, "dq"), _ptr(dk, io, s4, "dk"), _ptr(dv, io, s4, "dv"),
        _ptr(d_eta, f32, s3, "d_eta"), _ptr(d_beta, f32, s3, "d_beta"), _ptr(d_gamma, f32, s3, "d_gamma"),
        _table(dW_init, p, "dW_init"), _table(dM_init, p, "dM_init"), _row_table(d_row_norm, p, "d_row_norm"),
        _ptr(workspace, torch.uint8, None, "workspace"), workspace.numel() if workspace is not None else 0,
        int(states_saved), _stream_ptr(stream))
    if st != E2TTT_OK:
        raise E2TTTError(st, "e2ttt_chunk_bwd_normed")
    return st


def e2ttt_prepare_fwd(p, g, q_raw, k_raw, a_eta, a_beta, a_alpha, q, k, eta, beta, gamma, stream=None):
    """int e2ttt_prepare_fwd(...) of include/e2ttt.h.  Raises on error."""
    io = _io_torch_dtype(p)
    s4, s3 = (p.B, p.H, p.L, p.d), (p.B, p.H, p.L)
    f32 = torch.float32
    st = lib().e2ttt_prepare_fwd(
        ctypes.byref(p), ctypes.byref(g), _ptr(q_raw, io, s4, "q_raw"), _ptr(k_raw, io, s4, "k_raw"),
        _ptr(a_eta, f32, s3, "a_eta"), _ptr(a_beta, f32, s3, "a_beta"), _ptr(a_alpha, f32, s3, "a_alpha"),
        _ptr(q, io, s4, "q"), _ptr(k, io, s4, "k"), _ptr(eta, f32, s3, "eta"), _ptr(beta, f32, s3, "beta"),
        _ptr(gamma, f32, s3, "gamma"), _stream_ptr(stream))
    if st != E2TTT_OK:
        raise E2TTTError(st, "e2ttt_prepare_fwd")
    return st


def e2ttt_prepare_bwd(p, g, q_raw, k_raw, a_eta, a_beta, a_alpha, dq, dk, d_eta, d_beta, d_gamma, dq_raw, dk_raw,
                      da_eta, da_beta, da_alpha, stream=None):
    """int e2ttt_prepare_bwd(...) of include/e2ttt.h.  Raises on error."""
    io = _io_torch_dtype(p)
    s4, s3 = (p.B, p.H, p.L, p.d), (p.B, p.H, p.L)
    f32 = torch.float32
    st = lib().e2ttt_prepare_bwd(
        ctypes.byref(p), ctypes.byref(g), _ptr(q_raw, io, s4, "q_raw"), _ptr(k_raw, io, s4, "k_raw"),
        _ptr(a_eta, f32, s3, "a_eta"), _ptr(a_beta, f32, s3, "a_beta"), _ptr(a_alpha, f32, s3, "a_alpha"),
        _ptr(dq, io, s4, "dq"), _ptr(dk, io, s4, "dk"), _ptr(d_eta, f32, s3, "d_eta"), _ptr(d_beta, f32, s3, "d_beta"),
        _ptr(d_gamma, f32, s3, "d_gamma"), _ptr(dq_raw, io, s4, "dq_raw"), _ptr(dk_raw, io, s4, "dk_raw"),
        _ptr(da_eta, f32, s3, "da_eta"), _ptr(da_beta, f32, s3, "da_beta"), _ptr(da_alpha, f32, s3, "da_alpha"),
        _stream_ptr(stream))
    if st != E2TTT_OK:
        raise E2TTTError(st, "e2ttt_prepare_bwd")
    return st


def e2ttt_apply(p, q, W, o, stream=None):
    """int e2ttt_apply(...) of include/e2ttt.h: o = f_W(q) for p.L tokens per sequence, no update.  Raises on error."""
    io = _io_torch_dtype(p)
    s4 = (p.B, p.H, p.L, p.d)
    st = lib().e2ttt_apply(ctypes.byref(p), _ptr(q, io, s4, "q"), _table(W, p, "W"), _ptr(o, io, s4, "o"),
                           _stream_ptr(stream))
    if st != E2TTT_OK:
        raise E2TTTError(st, "e2ttt_apply")
    return st


def e2ttt_chunk_bwd(p, q, k, v, eta, beta, gamma, W_init, M_init, d_o, dW_final, dM_final, dq, dk, dv,
                    d_eta, d_beta, d_gamma, dW_init, dM_init, workspace, states_saved=0, stream=None):
    """int e2ttt_chunk_bwd(...) of include/e2ttt.h.  Raises on error."""
    io = _io_torch_dtype(p)
    s4, s3 = (p.B, p.H, p.L, p.d), (p.B, p.H, p.L)
    f32 = torch.float32
    st = lib().e2ttt_chunk_bwd(
        ctypes.byref(p), _ptr(q, io, s4, "q"), _ptr(k, io, s4, "k"), _ptr(v, io, s4, "v"),
        _ptr(eta, f32, s3, "eta"), _ptr(beta, f32, s3, "beta"), _ptr(gamma, f32, s3, "gamma"),
        _table(W_init, p, "W_init"), _table(M_init, p, "M_init"), _ptr(d_o, io, s4, "d_o"),
        _table(dW_final, p, "dW_final"), _table(dM_final, p, "dM_final"),
        _ptr(dq, io, s4, "dq"), _ptr(dk, io, s4, "dk"), _ptr(dv, io, s4, "dv"),
        _ptr(d_eta, f32, s3, "d_eta"), _ptr(d_beta, f32, s3, "d_beta"), _ptr(d_gamma, f32, s3, "d_gamma"),
        _table(dW_init, p, "dW_init"), _table(dM_init, p, "dM_init"),
        _ptr(workspace, torch.uint8, None, "workspace"), workspace.numel() if workspace is not None else 0,
        int(states_saved), _stream_ptr(stream))
    if st != E2TTT_OK:
        raise E2TTTError(st, "e2ttt_chunk_bwd")
    return st


def e2ttt_device_status(workspace, stream=None) -> int:
    """int e2ttt_device_status(...): waits for the stream and returns the device status word (0 = clean).
    workspace=None reads the word of the scratch array that e2ttt_chunk_fwd_noalloc uses on the current device."""
    word = ctypes.c_int(-1)
    wp = None if workspace is None else _ptr(workspace, torch.uint8, None, "workspace")
    st = lib().e2ttt_device_status(wp, _stream_ptr(stream), ctypes.byref(word))
    if st not in (E2TTT_OK, -8):
        raise E2TTTError(st, "e2ttt_device_status")
    return int(word.value)


def e2ttt_selftest_wait_timeout(workspace, limit_cycles: int, stream=None) -> int:
    """int e2ttt_selftest_wait_timeout(...): enqueues one CTA whose bounded wait runs out after limit_cycles."""
    st = lib().e2ttt_selftest_wait_timeout(_ptr(workspace, torch.uint8, None, "workspace"), workspace.numel(),
                                           int(limit_cycles), _stream_ptr(stream))
    if st != E2TTT_OK:
        raise E2TTTError(st, "e2ttt_selftest_wait_timeout")
    return st


E2TTT_NOALLOC_SCRATCH_BYTES = 8 << 20


def e2ttt_chunk_fwd_noalloc(p, q, k, v, eta, beta, gamma, W_init, M_init, o, W_final, M_final, stream=None):
    """int e2ttt_chunk_fwd_noalloc(...) of include/e2ttt.h: the forward for callers that cannot allocate a
    workspace (the scratch is a fixed array inside the library).  Raises on error, e.g. E2TTT_ERR_WORKSPACE
    when the shape needs more than E2TTT_NOALLOC_SCRATCH_BYTES."""
    io = _io_torch_dtype(p)
    s4, s3 = (p.B, p.H, p.L, p.d), (p.B, p.H, p.L)
    st = lib().e2ttt_chunk_fwd_noalloc(
        ctypes.byref(p), _ptr(q, io, s4, "q"), _ptr(k, io, s4, "k"), _ptr(v, io, s4, "v"),
        _ptr(eta, torch.float32, s3, "eta"), _ptr(beta, torch.float32, s3, "beta"),
        _ptr(gamma, torch.float32, s3, "gamma"), _table(W_init, p, "W_init"), _table(M_init, p, "M_init"),
        _ptr(o, io, s4, "o"), _table(W_final, p, "W_final"), _table(M_final, p, "M_final"), _stream_ptr(stream))
    if st != E2TTT_OK:
        raise E2TTTError(st, "e2ttt_chunk_fwd_noalloc")
    return st
