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


def _free_bytes():
    torch.cuda.synchronize()
    return torch.cuda.mem_get_info()[0]


def _both(L, gfw=None, fx=None):
    ws, xs = layer_scales(L)
    gfw = gfw or (fpq.E4M3 if L.wfmt == "e4m3" else fpq.E2M1)
    fx = fx or fpq.E4M3
    _, prep = gpu_prepare(L, ws)
    x = torch.from_numpy(L.x).cuda()
    bias = torch.from_numpy(L.bias).cuda()
    wsd = torch.from_numpy(ws).cuda()
    y_ref = fpq.fpq_linear(x, prep, wsd, xs, fx, gfw, bias, L.N)
    y = torch.full((L.M, L.N), float("nan"), dtype=torch.float32, device="cuda")
    fpq.fpq_linear_static(x, prep, wsd, xs, fx, gfw, bias, y)      # the first call on a device resolves the array
    y.fill_(float("nan"))
    # the driver's own count of free device memory: it moves for ANY allocation in this process, whoever made it
    # (torch's counters only see torch's allocator)
    before = _free_bytes()
    fpq.fpq_linear_static(x, prep, wsd, xs, fx, gfw, bias, y)
    assert _free_bytes() == before
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


def test_a_handful_of_rows_leaves_the_array_alone():
    # M <= 8 runs on the CUDA cores in one pass over the weights: no intermediate codes at all
    L = I.draw(I.linear_layer("few", 4, 320, 1280, "e2m1", rounding=True), 12, 20, "normal", 0.02, True)
    y, y_ref, ws, xs = _both(L)
    assert np.array_equal(y, y_ref)
    yo, ab = oracle_layer(L, ws, xs)
    assert_close(y, yo, ab)


def test_formats_that_need_more_scratch_per_element():
    """Weights prepared as two tensor-core terms keep two copies of the activation codes, so they reach the end of
    the array at half the documented size: within it the result equals fpq_linear's, beyond it the answer is
    FPQ_ERR_WORKSPACE (the size test on M x K has passed), never a partial result."""
    e3m4 = fpq.E3M4
    M, K, N = 300, 320, 200
    x = torch.randn(M, K, device="cuda")
    w = torch.randn(N, K, device="cuda") * 0.02
    ws = (w.abs().amax(dim=1) / fpq.fpq_format_max(e3m4)).contiguous()
    prep = fpq.fpq_prepare_weight(fpq.fpq_quantize_weight(w, ws, e3m4, None), e3m4, fpq.LINEAR, N, K)
    xs = float(x.abs().max()) / 448.0
    y_ref = fpq.fpq_linear(x, prep, ws, xs, fpq.E4M3, e3m4, None, N)
    y = torch.full((M, N), float("nan"), device="cuda")
    fpq.fpq_linear_static(x, prep, ws, xs, fpq.E4M3, e3m4, None, y)
    assert fpq.fpq_read_status() == fpq.OK
    assert torch.equal(y, y_ref)
    # 6000 x 1024 codes fit the array once (6 MiB of 8) but not twice
    Lb = fpq.lib()
    p = torch.zeros(256, dtype=torch.float32, device="cuda").data_ptr()
    assert 6000 * 1024 <= fpq.STATIC_SCRATCH_BYTES < 2 * 6000 * 1024
    assert Lb.fpq_linear_static(p, p, p, 1.0, fpq.E4M3.c(), e3m4.c(), None, p, 6000, 64, 1024, None) == fpq.ERR_WORKSPACE
    # activations in a format the tensor cores have no type for run on the CUDA cores with FP32 scratch:
    # a small problem fits, a larger one that passes the M x K test does not
    e2m5 = fpq.E2M5
    xs5 = float(x.abs().max()) / fpq.fpq_format_max(e2m5)
    w8 = (w.abs().amax(dim=1) / 448.0).contiguous()
    prep8 = fpq.fpq_prepare_weight(fpq.fpq_quantize_weight(w, w8, fpq.E4M3, None), fpq.E4M3, fpq.LINEAR, N, K)
    y_ref = fpq.fpq_linear(x, prep8, w8, xs5, e2m5, fpq.E4M3, None, N)
    y.fill_(float("nan"))
    fpq.fpq_linear_static(x, prep8, w8, xs5, e2m5, fpq.E4M3, None, y)
    assert fpq.fpq_read_status() == fpq.OK
    assert torch.equal(y, y_ref)
    assert fpq.fpq_linear_workspace_size(6000, 64, 1024, e2m5, fpq.E4M3) > fpq.STATIC_SCRATCH_BYTES
    assert Lb.fpq_linear_static(p, p, p, 1.0, e2m5.c(), fpq.E4M3.c(), None, p, 6000, 64, 1024, None) == fpq.ERR_WORKSPACE
