"""Training-memory plan (Section 3.2 leaves it to the implementation): with e2ttt_params.ckpt_every = n >= 2 the forward
keeps the state of every n-th chunk only and the backward recomputes n chunk-start states at a time.  The arithmetic of
every chunk is unchanged, so the gradients must equal those of the keep-everything plan bit for bit whenever both plans
read states produced by the same kernel, and agree with the oracle's backward as before."""
import numpy as np
import pytest
import torch

from paper_2608_21308_b200 import binding as E
from paper_2608_21308_b200 import inputs
from tests import util
from tests.test_gpu_parity import check_backward

pytestmark = pytest.mark.gpu

MLP, SWIGLU = E.E2TTT_MLP_GELU, E.E2TTT_SWIGLU
TOL_F32, TOL_BF16 = 1e-4, 2e-2
GRADS = ("dq", "dk", "dv", "deta", "dbeta", "dgamma")


def same_bits(a, b, what):
    for n in GRADS:
        assert np.array_equal(a[n], b[n]), f"{what}: {n}"
    for i in range(len(a["dW"])):
        assert np.array_equal(a["dW"][i], b["dW"][i]), f"{what}: dW{i + 1}"
        assert np.array_equal(a["dM"][i], b["dM"][i]), f"{what}: dM{i + 1}"


@pytest.mark.parametrize("kind", [MLP, SWIGLU])
@pytest.mark.parametrize("every,L", [(3, 8 * 8 + 3), (2, 8 * 5), (4, 8 * 4), (16, 8 * 6)])
def test_segmented_backward_fp32_matches_the_oracle_and_the_keep_everything_plan(kind, every, L):
    """9 chunks with a ragged last one in segments of 3; an odd number of segments of 2; exactly one segment; a segment
    longer than the sequence."""
    r = inputs.paper_regime(inputs.Recipe(B=3, H=1, L=L, d=24, h=40, C=8, kind=kind, seed=31, m_std=0.002))
    x = inputs.generate(r, with_d_o=True, with_dstate=True)
    shape = dict(d=r.d, h=r.h, C=r.C, kind=kind, io="f32")
    ref = util.oracle_backward(x, r.C, kind)
    full = util.gpu_backward(x, **shape)
    check_backward(full, ref, TOL_F32, "every chunk kept")
    for saved in (False, True):
        got = util.gpu_backward(x, ckpt_every=every, via_saved_states=saved, **shape)
        check_backward(got, ref, TOL_F32, f"checkpoints every {every}, saved={saved}")
        same_bits(got, full, f"every {every}, saved={saved}")


@pytest.mark.parametrize("kind,d,h", [(MLP, 128, 512), (SWIGLU, 128, 384)])
def test_segmented_backward_bf16_tiled(kind, d, h):
    """bf16 I/O on the tensor-core any-shape kernels, 20 chunks in segments of 8 (8 + 8 + 4), paper-regime gates."""
    r = inputs.paper_regime(inputs.Recipe(B=2, H=1, L=64 * 20, d=d, h=h, C=64, kind=kind, io="bf16", seed=33, m_std=0.002))
    x = inputs.generate(r, with_d_o=True, with_dstate=True)
    shape = dict(d=d, h=h, C=64, kind=kind, io="bf16", impl=E.E2TTT_IMPL_TILED)
    full = util.gpu_backward(x, **shape)
    for saved in (False, True):
        got = util.gpu_backward(x, ckpt_every=8, via_saved_states=saved, **shape)
        same_bits(got, full, f"tiled, saved={saved}")


def test_fused_forward_writes_the_checkpoints_and_recomputes_the_segments():
    """Training flow at the benchmark shape: the fused forward keeps every 4th chunk-start state and the backward has the
    same fused kernel recompute the others, restarted from its own fp32 checkpoint: bit for bit the gradients of the flow
    in which the fused forward kept every state, of the flow in which nothing was saved (everything recomputed), and, on
    the last segment, of a backward that is handed the fused kernel's own state after 4 chunks as its initial state."""
    r = inputs.config(2, heads=[3, 40])
    shape = dict(d=r.d, h=r.h, C=r.C, kind=r.kind, io="bf16")
    x2, _ = util.teacher_forced_windows(r, 8, window=8, with_grads=True)   # 8 chunks per call, 2 segments of 4
    a = util.gpu_backward(x2, via_saved_states=True, ckpt_every=4, **shape)
    b = util.gpu_backward(x2, via_saved_states=True, **shape)
    c = util.gpu_backward(x2, via_saved_states=False, ckpt_every=4, **shape)
    d = util.gpu_backward(x2, via_saved_states=False, **shape)
    same_bits(a, b, "checkpoints every 4 vs every state kept")
    same_bits(a, c, "saved checkpoints vs recomputed checkpoints")
    same_bits(a, d, "vs everything recomputed in one go")
    x4 = {n: (np.ascontiguousarray(v[:, :4 * 64]) if not isinstance(v, list) else v) for n, v in x2.items()}
    st4, _ = util.gpu_forward(x4, impl=E.E2TTT_IMPL_TCGEN05, **shape)
    x_tail = {n: (np.ascontiguousarray(v[:, 4 * 64:]) if not isinstance(v, list) else v) for n, v in x2.items()}
    x_tail["W"], x_tail["M"] = st4["W"], st4["M"]
    tail = util.gpu_backward(x_tail, via_saved_states=False, **shape)
    for n in GRADS:
        assert np.array_equal(a[n][:, 4 * 64:], tail[n]), n
    # the any-shape kernels on the same flow (two-term bf16 operands): close to the fused states' gradients, not equal
    t = util.gpu_backward(x2, via_saved_states=False, ckpt_every=4, impl=E.E2TTT_IMPL_TILED, **shape)
    for n in GRADS:
        assert util.rel_err(a[n], t[n]) <= 0.15, n   # 8 chunks free-running under the benchmark gates (a chaotic map)


def test_padded_shape_short_chunks_ragged_tail_and_checkpoints_together():
    """Config 1's shape (d = 64, h = 256: the fused kernel's zero-padded instantiation) with chunks of 32 tokens, a
    ragged last chunk and checkpoints every 2 chunks: forward against the oracle, and the three memory plans of the
    backward bit for bit."""
    r = inputs.paper_regime(inputs.Recipe(B=3, H=1, L=5 * 32 + 9, d=64, h=256, C=32, kind=MLP, io="bf16", seed=41, m_std=0.002))
    x = inputs.generate(r, with_d_o=True, with_dstate=True)
    shape = dict(d=64, h=256, C=32, kind=MLP, io="bf16")
    ref = util.oracle_forward(x, 32, MLP)
    got, hd = util.gpu_forward(x, **shape)
    assert hd["ws"].numel() == 256 and E.e2ttt_device_status(hd["ws"]) == 0
    from tests.test_gpu_parity import check_forward
    check_forward(got, ref, TOL_BF16, "padded shape, C = 32, ragged")
    a = util.gpu_backward(x, via_saved_states=True, **shape)
    b = util.gpu_backward(x, via_saved_states=True, ckpt_every=2, **shape)
    c = util.gpu_backward(x, via_saved_states=False, ckpt_every=4, **shape)
    same_bits(a, b, "padded: every state vs checkpoints every 2")
    same_bits(a, c, "padded: every state vs recomputed checkpoints every 4")
    check_backward(a, util.oracle_backward(x, 32, MLP), 3 * TOL_BF16, "padded shape backward, 6 chunks free-running")


@pytest.mark.parametrize("cfg", [2, 3])
def test_full_size_training_flow_memory_plans_agree(cfg):
    """The launch configurations bench.py --backward times (B=4, H=16, L=4096, 64 chunks; GELU-MLP and SwiGLU): forward
    with saved states + backward, with every state kept and with checkpoints every 8 chunks (8 segments, each recomputed
    by the fused forward): gradients finite and the same bits.  (The SwiGLU run takes the paper's gate regime: under the
    benchmark gates its adjoint leaves the bf16 range within 64 free-running chunks.)"""
    r = inputs.config(cfg) if cfg == 2 else inputs.paper_regime(inputs.config(cfg))
    x = inputs.generate(r, with_d_o=True, with_dstate=True)
    shape = dict(d=r.d, h=r.h, C=r.C, kind=r.kind, io="bf16")
    a = util.gpu_backward(x, via_saved_states=True, **shape)
    b = util.gpu_backward(x, via_saved_states=True, ckpt_every=8, **shape)
    for n in GRADS:
        assert np.isfinite(a[n]).all(), n
    same_bits(a, b, "full size: every state kept vs checkpoints every 8")
