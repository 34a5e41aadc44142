"""The forward entry point for callers that cannot allocate device memory (e2ttt_chunk_fwd_noalloc).

Some users of the library are handed their input and output buffers and nothing else: a plugin inside
an application that owns the memory pool, or a loop that must not call the allocator once it runs.
They cannot provide the workspace e2ttt_chunk_fwd wants, so the library carries a fixed scratch array
for them.  This test drives that entry point through the C ABI twice in a row, with different inputs,
and checks each result against the ordinary entry point: the second call finds the first call's
leftovers in the shared scratch and must not care.  Collected last on purpose (file name), and it must
pass alone in a fresh process as well as after every other test.
"""
import numpy as np
import pytest
import torch

from paper_2608_21308_b200 import binding as E
from paper_2608_21308_b200 import inputs
from tests import util

pytestmark = pytest.mark.gpu

TOL = 1e-4  # the fp32-I/O tolerance of the parity tests


def _run_both(seed, L):
    r = inputs.Recipe(B=1, H=2, L=L, d=64, h=256, C=16, kind=inputs.KIND_MLP, io="f32", seed=seed, m_std=0.01)
    x = inputs.generate(r)
    ref, hd = util.gpu_forward(x, d=r.d, h=r.h, C=r.C, kind=r.kind, io="f32")
    # the same device tensors and parameters as the ordinary call (the helper lays the 2 sequences out as B=2, H=1)
    p = hd["p"]
    o = torch.full_like(hd["q"], float("nan"))
    Wf = [torch.full_like(w, float("nan")) for w in hd["W"]]
    Mf = [torch.full_like(w, float("nan")) for w in hd["W"]]
    before = torch.cuda.memory_allocated()
    E.e2ttt_chunk_fwd_noalloc(p, hd["q"], hd["k"], hd["v"], hd["eta"], hd["beta"], hd["gamma"], hd["W"], hd["M"],
                              o, Wf, Mf)
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == before
    N = x["q"].shape[0]
    got = {"o": o.cpu().numpy().reshape(N, L, r.d), "W": [w.cpu().numpy()[:, 0] for w in Wf],
           "M": [m.cpu().numpy()[:, 0] for m in Mf]}
    return got, ref


def test_noalloc_forward_matches_the_ordinary_entry_point_twice_in_a_row():
    for seed, L in ((21, 64), (22, 48)):  # second call: other inputs, other length, same scratch
        got, ref = _run_both(seed, L)
        assert util.rel_err(got["o"], ref["o"]) <= TOL
        for i in range(2):
            assert util.rel_err(got["W"][i], ref["W"][i]) <= TOL
            assert util.rel_err(got["M"][i], ref["M"][i]) <= TOL
        assert np.isfinite(got["o"]).all()


def test_noalloc_forward_matches_the_oracle_and_reports_its_status():
    """The entry point stands on its own: compared with the fp64 oracle directly, and its device status word (kept in
    the library's scratch array, read with workspace = None) is clean afterwards."""
    r = inputs.Recipe(B=1, H=2, L=64, d=64, h=256, C=16, kind=inputs.KIND_MLP, io="f32", seed=23, m_std=0.01)
    x = inputs.generate(r)
    got, _ = _run_both(23, 64)
    ref = util.oracle_forward(x, r.C, r.kind)
    assert util.rel_err(got["o"], ref["o"]) <= TOL
    for i in range(2):
        assert util.rel_err(got["W"][i], ref["W"][i]) <= TOL
        assert util.rel_err(got["M"][i], ref["M"][i]) <= TOL
    assert E.e2ttt_device_status(None) == 0


def test_noalloc_refuses_shapes_beyond_its_fixed_scratch():
    p = E.make_params(4, 16, 64, 128, 512, 64, io_dtype=E.E2TTT_BF16, impl=E.E2TTT_IMPL_SIMT)  # SIMT scratch: ~100 MB
    assert E.e2ttt_workspace_bytes(p, 0) > E.E2TTT_NOALLOC_SCRATCH_BYTES
    t4 = torch.zeros(4, 16, 64, 128, device="cuda", dtype=torch.bfloat16)
    t3 = torch.zeros(4, 16, 64, device="cuda")
    W = [torch.zeros(4, 16, 512, 128, device="cuda"), torch.zeros(4, 16, 128, 512, device="cuda")]
    o = torch.full_like(t4, 3.0)
    with pytest.raises(E.E2TTTError) as ei:
        E.e2ttt_chunk_fwd_noalloc(p, t4, t4, t4, t3, t3, t3, W, None, o, W, W)
    assert ei.value.status == -5
    torch.cuda.synchronize()
    assert float(o.float().min()) == 3.0
