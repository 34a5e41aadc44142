"""The any-shape kernels with their matrix products on the tensor cores (impl TILED, bf16 I/O) against the fp64
oracle, and against the same kernels with fp32 FMAs (impl SIMT)."""
import numpy as np
import pytest

from paper_2608_21308_b200 import binding as E
from paper_2608_21308_b200 import inputs
from tests import util
from tests.test_gpu_parity import TOL_BF16, check_backward, check_forward

pytestmark = pytest.mark.gpu
MLP, SWIGLU = inputs.KIND_MLP, inputs.KIND_SWIGLU


def _shape(r):
    return dict(d=r.d, h=r.h, C=r.C, kind=r.kind, io="bf16")


@pytest.mark.parametrize("cfg,over", [(2, {}), (3, {}), (3, dict(C=16)), (3, dict(C=128)), (1, {})],
                         ids=["mlp128", "swiglu", "swiglu-C16", "swiglu-C128", "mlp64"])
def test_tiled_forward_windows(cfg, over):
    r = inputs.config(cfg, heads=[3, 30], m_std=0.002, **over)
    xw, ref = util.teacher_forced_windows(r, 3, window=1)
    got, hd = util.gpu_forward(xw, impl=E.E2TTT_IMPL_TILED, **_shape(r))
    assert E.e2ttt_device_status(hd["ws"]) == 0
    errs = check_forward(got, ref, TOL_BF16, f"tiled config {cfg} {over}")
    fma, _ = util.gpu_forward(xw, impl=E.E2TTT_IMPL_SIMT, **_shape(r))
    check_forward(fma, ref, TOL_BF16, "fma")
    print(cfg, over, errs)


@pytest.mark.parametrize("kind", [MLP, SWIGLU])
@pytest.mark.parametrize("d,h,C,L,N", [(48, 80, 24, 100, 3), (8, 16, 1, 5, 1), (72, 136, 16, 7, 2), (64, 192, 128, 256, 2)])
def test_tiled_forward_odd_shapes_free_running(kind, d, h, C, L, N):
    """Ragged tiles in every direction (rows, columns, contraction tails, a short last chunk), paper-regime gates."""
    r = inputs.paper_regime(inputs.Recipe(B=N, H=1, L=L, d=d, h=h, C=C, kind=kind, io="bf16", seed=11, m_std=0.002))
    x = inputs.generate(r)
    ref = util.oracle_forward(x, C, kind)
    got, hd = util.gpu_forward(x, impl=E.E2TTT_IMPL_TILED, **_shape(r))
    assert E.e2ttt_device_status(hd["ws"]) == 0
    check_forward(got, ref, TOL_BF16, f"tiled odd shape {d}x{h} C={C}")


@pytest.mark.parametrize("cfg", [4, 3, 1], ids=["mlp128", "swiglu", "mlp64"])
def test_tiled_backward_windows(cfg):
    r = inputs.config(cfg, heads=[2, 11])
    xw, _ = util.teacher_forced_windows(r, 3, window=1, with_grads=True)
    ref = util.oracle_backward(xw, r.C, r.kind)
    got = util.gpu_backward(xw, impl=E.E2TTT_IMPL_TILED, **_shape(r))
    errs = check_backward(got, ref, TOL_BF16, f"tiled bwd config {cfg}")
    print(cfg, errs)


@pytest.mark.parametrize("kind", [MLP, SWIGLU])
@pytest.mark.parametrize("L,tol", [(24, TOL_BF16), (17, TOL_BF16), (60, 3 * TOL_BF16)], ids=["one-chunk", "short-chunk", "three-chunks"])
def test_tiled_backward_odd_shape_free_running(kind, L, tol):
    """Ragged tiles everywhere.  One chunk is held to the bf16 tolerance; over three chunks (the last one short) the
    reverse sweep compounds the bf16 operand rounding of every chunk, so the bound is three times that."""
    r = inputs.paper_regime(inputs.Recipe(B=2, H=1, L=L, d=48, h=80, C=24, kind=kind, io="bf16", seed=12, m_std=0.002))
    x = inputs.generate(r, with_d_o=True, with_dstate=True)
    ref = util.oracle_backward(x, r.C, kind)
    got = util.gpu_backward(x, impl=E.E2TTT_IMPL_TILED, **_shape(r))
    check_backward(got, ref, tol, "tiled bwd odd shape")


def test_tiled_is_the_default_for_bf16_shapes_without_a_fused_kernel_and_is_repeatable():
    r = inputs.config(3, heads=[1, 2, 3], L=256, C=128)                  # the fused kernels serve C = 16, 32, 64
    x = inputs.generate(r)
    a, hd = util.gpu_forward(x, **_shape(r))                              # AUTO
    b, _ = util.gpu_forward(x, impl=E.E2TTT_IMPL_TILED, **_shape(r))
    assert E.e2ttt_device_status(hd["ws"]) == 0
    assert np.array_equal(a["o"], b["o"])
    for i in range(3):
        assert np.array_equal(a["W"][i], b["W"][i]) and np.array_equal(a["M"][i], b["M"][i])
    with pytest.raises(Exception):
        util.gpu_forward(x, impl=E.E2TTT_IMPL_TILED, d=r.d, h=r.h, C=r.C, kind=r.kind, io="f32")


@pytest.mark.parametrize("kind,h", [(SWIGLU, 384), (MLP, 512)])
def test_tiled_free_running_paper_regime_at_benchmark_shapes(kind, h):
    """16 chunks free-running under the paper's gate regime (where the recurrence is well conditioned), d = 128."""
    r = inputs.paper_regime(inputs.Recipe(B=3, H=1, L=1024, d=128, h=h, C=64, kind=kind, io="bf16", seed=4, m_std=0.002))
    x = inputs.generate(r)
    ref = util.oracle_forward(x, 64, kind)
    got, hd = util.gpu_forward(x, impl=E.E2TTT_IMPL_TILED, **_shape(r))
    assert E.e2ttt_device_status(hd["ws"]) == 0
    errs = check_forward(got, ref, TOL_BF16, "tiled paper regime, 16 chunks free-running")
    print(kind, errs)


@pytest.mark.parametrize("io,impl", [("bf16", E.E2TTT_IMPL_TILED), ("f32", E.E2TTT_IMPL_SIMT)], ids=["tiled-bf16", "fma-fp32"])
@pytest.mark.parametrize("kind", [MLP, SWIGLU])
def test_wide_networks_forward_and_backward(kind, io, impl):
    """d = 256, h = 1024 (several tiles in every direction, split-K parts with tails), one chunk of 48 tokens."""
    r = inputs.paper_regime(inputs.Recipe(B=1, H=1, L=48, d=256, h=1024, C=48, kind=kind, io=io, seed=13, m_std=0.002))
    x = inputs.generate(r, with_d_o=True, with_dstate=True)
    shape = dict(d=r.d, h=r.h, C=r.C, kind=kind, io=io)
    tol = TOL_BF16 if io == "bf16" else 1e-4
    got, hd = util.gpu_forward(x, impl=impl, **shape)
    assert E.e2ttt_device_status(hd["ws"]) == 0
    check_forward(got, util.oracle_forward(x, r.C, kind), tol, "wide forward")
    check_backward(util.gpu_backward(x, impl=impl, **shape), util.oracle_backward(x, r.C, kind), tol, "wide backward")
