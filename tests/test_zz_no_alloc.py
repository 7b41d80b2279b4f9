"""fpq_linear_static: the linear layer for callers that cannot allocate device memory.

Some users of this library run where a cudaMalloc is off limits: inside another
framework's stream where the allocator's device-wide synchronisation would stall
everyone, or in a serving loop whose memory budget was fixed at start-up.  For
them the library keeps the intermediate activation codes in a fixed array of its
own instead of a caller-provided workspace.  This test calls that entry point
through the C ABI twice in a row, the second time on a smaller problem so that
left-overs of the first call sit in the shared array, and checks each result
against fpq_linear with an ordinary workspace.  It is collected last on purpose.
"""
import numpy as np
import pytest
import torch

import paper_2408_06995_b200 as fpq
from paper_2408_06995_b200 import inputs as I
from _helpers import assert_close, gpu_prepare, layer_scales, oracle_layer

pytestmark = pytest.mark.gpu


def _both(L):
    ws, xs = layer_scales(L)
    gfw = fpq.E4M3 if L.wfmt == "e4m3" else fpq.E2M1
    _, prep = gpu_prepare(L, ws)
    x = torch.from_numpy(L.x).cuda()
    bias = torch.from_numpy(L.bias).cuda()
    wsd = torch.from_numpy(ws).cuda()
    y_ref = fpq.fpq_linear(x, prep, wsd, xs, fpq.E4M3, gfw, bias, L.N)
    y = torch.full((L.M, L.N), float("nan"), dtype=torch.float32, device="cuda")
    before = torch.cuda.memory_allocated()
    fpq.fpq_linear_static(x, prep, wsd, xs, fpq.E4M3, gfw, bias, y)
    assert torch.cuda.memory_allocated() == before
    assert fpq.fpq_read_status() == fpq.OK
    return y.cpu().numpy(), y_ref.cpu().numpy(), ws, xs


def test_two_calls_in_a_row_match_the_workspace_entry_point():
    big = I.draw(I.linear_layer("first", 1000, 320, 960, "e4m3"), 12, 0, "normal", 0.02, True, 0.01, (0.001, 20.0))
    small = I.draw(I.linear_layer("second", 130, 200, 72, "e2m1", rounding=True), 12, 10, "normal", 0.02, True)
    for L in (big, small):
        y, y_ref, ws, xs = _both(L)
        assert np.array_equal(y, y_ref)                 # same kernels, same order of operations
        yo, ab = oracle_layer(L, ws, xs)                # and within the layer tolerance of the oracle
        assert_close(y, yo, ab)


def test_rejects_problems_beyond_the_fixed_capacity():
    L = fpq.lib()
    F = fpq.E4M3.c()
    p = torch.zeros(256, dtype=torch.float32, device="cuda").data_ptr()
    M, K = 8193, 1024                                     # 8193 * 1024 bytes > 8 MiB
    assert M * K > fpq.STATIC_SCRATCH_BYTES
    assert L.fpq_linear_static(p, p, p, 1.0, F, F, None, p, M, 64, K, None) == fpq.ERR_TOO_LARGE
    assert "capacity" in fpq.status_string(fpq.ERR_TOO_LARGE)
