"""The device-side failure path, exercised without failing anything: a bounded wait that runs out is reported
through the status word and leaves the context usable."""
import numpy as np
import pytest
import torch

from paper_2608_21308_b200 import binding as E
from paper_2608_21308_b200 import inputs
from tests import util

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_sets_the_status_word_and_the_context_stays_usable():
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    E.e2ttt_selftest_wait_timeout(ws, 300_000)           # ~0.15 ms: nobody ever signals the barrier it waits on
    word = E.e2ttt_device_status(ws)                      # synchronises
    assert word == 900                                    # the code of the first wait that gave up
    st = E.lib().e2ttt_device_status(ws.data_ptr(), None, __import__("ctypes").byref(__import__("ctypes").c_int()))
    assert st == -8 and E.e2ttt_status_string(st) == "a bounded device-side wait gave up"
    # nothing trapped: the next real call on the same context runs clean
    r = inputs.config(2, heads=[1], L=128)
    x = inputs.generate(r)
    got, hd = util.gpu_forward(x, impl=E.E2TTT_IMPL_TCGEN05, d=r.d, h=r.h, C=r.C, kind=r.kind, io="bf16")
    assert E.e2ttt_device_status(hd["ws"]) == 0 and np.isfinite(got["o"]).all()
    # a clean launch on the same workspace clears the word again
    E.e2ttt_selftest_wait_timeout(ws, 200_000)
    assert E.e2ttt_device_status(ws) == 900
