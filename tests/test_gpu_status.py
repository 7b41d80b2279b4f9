"""The device status word and the bounded waits (failure detection without a GPU fault): a wait that
nothing satisfies runs out after its limit, the kernel records ERR_TIMEOUT and returns, and the context
stays usable for the next layer call."""
import numpy as np
import pytest
import torch

import paper_2408_06995_b200 as fpq
from paper_2408_06995_b200 import inputs as I
from _helpers import assert_close, gpu_layer, layer_scales, oracle_layer

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    assert fpq.fpq_read_status() == fpq.OK
    fpq.fpq_selftest_bounded_wait(100_000)           # 1e5 cycles: about 50 microseconds
    assert fpq.fpq_read_status() == fpq.ERR_TIMEOUT
    assert fpq.fpq_read_status() == fpq.OK           # reading clears the word
    # the next layer call is unaffected
    L = I.draw(I.conv_layer("after", 2, 128, 32, 32, 128, 3, wfmt="e4m3", rounding=True), 21, 0, "silu", 0.03, True)
    ws, xs = layer_scales(L)
    y = gpu_layer(L, ws, xs)
    yr, ab = oracle_layer(L, ws, xs)
    assert_close(y, yr, ab)


def test_a_timeout_is_not_hidden_by_a_nan_input():
    x = torch.randn(4096, device="cuda")
    x[17] = float("nan")
    codes = fpq.fpq_quantize_act(x, 0.01, fpq.E4M3)
    torch.cuda.synchronize()
    fpq.fpq_selftest_bounded_wait(50_000)
    fpq.fpq_quantize_act(x, 0.01, fpq.E4M3)          # a second NaN event after the time-out
    assert fpq.fpq_read_status() == fpq.ERR_TIMEOUT  # the more serious event wins, whatever the order
    assert fpq.fpq_read_status() == fpq.OK
    assert int(codes[17]) == 0
    fpq.fpq_quantize_act(x, 0.01, fpq.E4M3)
    assert fpq.fpq_read_status() == fpq.ERR_NAN_INPUT
