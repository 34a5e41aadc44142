"""Host-side tests of the C ABI that need no GPU: the library loads, exports every declared symbol,
and rejects bad arguments before touching a device."""
import ctypes
import os
import re

import pytest

from paper_2608_21308_b200 import build as libbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    libbuild.build()
    from paper_2608_21308_b200 import binding
    return binding.lib()


def declared_symbols():
    names = []
    inc = os.path.join(ROOT, "include")
    for fn in sorted(os.listdir(inc)):
        if fn.endswith(".h"):
            text = open(os.path.join(inc, fn)).read()
            names += re.findall(r"E2TTT_API\s+[\w\s\*]+?\b(e2ttt_\w+)\s*\(", text)
    return names


def test_every_declared_symbol_is_exported(L):
    names = declared_symbols()
    assert {"e2ttt_chunk_fwd", "e2ttt_chunk_bwd", "e2ttt_workspace_bytes"} <= set(names)
    for n in names:
        assert hasattr(L, n), n


def test_status_strings_and_version(L):
    from paper_2608_21308_b200 import binding as E
    assert E.e2ttt_status_string(0) == "ok"
    for s in range(-8, 0):
        assert E.e2ttt_status_string(s) not in ("ok", "unknown status")
    assert E.e2ttt_status_string(-99) == "unknown status"
    assert E.e2ttt_version() >= 100


def test_matrix_shapes_follow_the_two_networks(L):
    from paper_2608_21308_b200 import binding as E
    assert E.e2ttt_num_matrices(E.E2TTT_MLP_GELU) == 2 and E.e2ttt_num_matrices(E.E2TTT_SWIGLU) == 3
    assert E.e2ttt_num_matrices(7) == 0
    assert [E.e2ttt_matrix_shape(E.E2TTT_MLP_GELU, 64, 256, i) for i in range(2)] == [(256, 64), (64, 256)]
    assert [E.e2ttt_matrix_shape(E.E2TTT_SWIGLU, 128, 384, i) for i in range(3)] == [(384, 128), (384, 128), (128, 384)]
    with pytest.raises(E.E2TTTError):
        E.e2ttt_matrix_shape(E.E2TTT_MLP_GELU, 64, 256, 2)


def test_workspace_sizes(L):
    from paper_2608_21308_b200 import binding as E
    p = E.make_params(1, 1, 256, 64, 256, 16)
    a = E.e2ttt_workspace_bytes(p, 0)
    b = E.e2ttt_workspace_bytes(p, 1)
    assert 0 < a < b
    # saved states: (W, M) of 2 matrices per chunk, fp64 internally for fp32 I/O
    assert b - a >= 16 * 2 * 2 * 64 * 256 * 8
    p2 = E.make_params(2, 3, 256, 64, 256, 16)
    assert E.e2ttt_workspace_bytes(p2, 0) - 256 == 6 * (a - 256)   # 256-byte status block + per-sequence scratch
    pb = E.make_params(1, 1, 256, 64, 256, 16, io_dtype=E.E2TTT_BF16, impl=E.E2TTT_IMPL_SIMT)
    assert (E.e2ttt_workspace_bytes(pb, 0) - 256) * 2 == a - 256
    pb.impl = E.E2TTT_IMPL_AUTO            # bf16, d = 64, h = 256, C = 16: the fused kernel serves it
    assert E.e2ttt_workspace_bytes(pb, 0) == 256
    # the tensor-core forward keeps all state on chip: only the status block
    pt = E.make_params(4, 16, 4096, 128, 512, 64, io_dtype=E.E2TTT_BF16)
    assert E.e2ttt_workspace_bytes(pt, 0) == 256
    assert E.e2ttt_workspace_bytes(pt, 1) > 256
    pt.impl = E.E2TTT_IMPL_SIMT
    assert E.e2ttt_workspace_bytes(pt, 0) > 256


def test_checkpoints_every_n_chunks_shrink_the_workspace_and_are_refused_by_the_normed_calls(L):
    from paper_2608_21308_b200 import binding as E
    kw = dict(io_dtype=E.E2TTT_BF16)
    full = E.make_params(4, 16, 32768, 128, 512, 64, **kw)
    seg = E.make_params(4, 16, 32768, 128, 512, 64, ckpt_every=32, **kw)
    a, b = E.e2ttt_workspace_bytes(full, 1), E.e2ttt_workspace_bytes(seg, 1)
    per_state = 64 * 4 * 128 * 512 * 4  # all sequences, (W1, W2, M1, M2), fp32
    assert a > 513 * per_state
    assert (16 + 1 + 32 + 1) * per_state < b < (16 + 1 + 32 + 1 + 12) * per_state
    assert E.e2ttt_workspace_bytes(full, 0) == E.e2ttt_workspace_bytes(seg, 0) == 256  # forward only: unchanged
    one = E.make_params(4, 16, 32768, 128, 512, 64, ckpt_every=1, **kw)
    assert E.e2ttt_workspace_bytes(one, 1) == a
    with pytest.raises(E.E2TTTError) as ei:
        E.e2ttt_workspace_bytes_normed(seg, 1)
    assert ei.value.status == -2


@pytest.mark.parametrize("field,value,status", [
    ("B", 0, -2), ("L", -1, -2), ("C", 0, -2), ("C", 513, -2), ("d", 0, -2), ("h", 100000, -2),
    ("kind", 2, -2), ("io_dtype", 5, -3), ("impl", 9, -3), ("impl", 2, -2), ("ckpt_every", -1, -2),
])
def test_bad_parameters_are_rejected(L, field, value, status):
    from paper_2608_21308_b200 import binding as E
    p = E.make_params(1, 1, 64, 16, 32, 16)
    setattr(p, field, value)
    n = ctypes.c_size_t()
    assert L.e2ttt_workspace_bytes(ctypes.byref(p), 0, ctypes.byref(n)) == status


def test_null_alignment_and_workspace_errors_come_before_any_device_use(L):
    from paper_2608_21308_b200 import binding as E
    p = E.make_params(1, 1, 64, 16, 32, 16)
    vp = ctypes.c_void_p
    good = vp(0x10000)  # never dereferenced: validation fails first
    tab2 = (vp * 2)(0x10000, 0x20000)
    need = E.e2ttt_workspace_bytes(p, 0)

    def fwd(q=good, W=tab2, ws=vp(0x100000), nbytes=need, o=good, M=None):
        return L.e2ttt_chunk_fwd(ctypes.byref(p), q, good, good, good, good, good, W, M, o, tab2, tab2, ws,
                                 nbytes, 0, None)

    assert fwd(q=None) == -1
    assert fwd(W=None) == -1
    assert fwd(W=(vp * 2)(0x10000, None)) == -1
    assert fwd(M=(vp * 2)(None, 0x10000)) == -1
    assert fwd(q=vp(0x10004)) == -4
    assert fwd(ws=None) == -5
    assert fwd(nbytes=need - 1) == -5
    assert fwd(ws=vp(0x100010)) == -4
    assert L.e2ttt_chunk_fwd(None, good, good, good, good, good, good, tab2, None, good, tab2, tab2,
                             vp(0x100000), need, 0, None) == -1
    # backward: NULL gradient outputs are refused
    args2 = [good] * 6 + [tab2, None, good, None, None, None] + [good] * 5 + [tab2, tab2, vp(0x100000), 1 << 30, 0, None]
    assert L.e2ttt_chunk_bwd(ctypes.byref(p), *args2) == -1


def test_binding_refuses_host_tensors(L):
    import torch
    from paper_2608_21308_b200 import binding as E
    p = E.make_params(1, 1, 16, 8, 16, 16)
    t = torch.zeros(1, 1, 16, 8)
    with pytest.raises(TypeError):
        E.e2ttt_chunk_fwd(p, t, t, t, t, t, t, [t, t], None, t, [t, t], [t, t], torch.zeros(8, dtype=torch.uint8))


def test_selftest_entry_point_validates_before_any_device_use(L):
    vp = ctypes.c_void_p
    f = L.e2ttt_selftest_wait_timeout
    f.argtypes = [vp, ctypes.c_size_t, ctypes.c_longlong, vp]
    assert f(None, 256, 1000, None) == -1
    assert f(vp(0x100000), 128, 1000, None) == -5
    assert f(vp(0x100010), 256, 1000, None) == -4
    assert f(vp(0x100000), 256, 0, None) == -2
    assert f(vp(0x100000), 256, 3_000_000_000, None) == -2


def test_device_status_of_the_noalloc_scratch_before_any_call_is_clean(L):
    word = ctypes.c_int(-1)
    assert L.e2ttt_device_status(None, None, ctypes.byref(word)) == 0 and word.value == 0
    assert L.e2ttt_device_status(None, None, None) == -1
