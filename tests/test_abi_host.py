"""CPU-side checks of the C-ABI library: it loads, exports every declared symbol,
and rejects what the host can detect before touching the GPU."""
import ctypes
import os
import re

import pytest

import paper_2408_06995_b200 as fpq
from paper_2408_06995_b200 import build as fpq_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    fpq_build.build()
    return fpq.lib()


def test_exports_every_declared_symbol(L):
    header = open(os.path.join(ROOT, "include", "fpq.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(fpq_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations found"
    assert declared == set(fpq.EXPORTS)
    for name in declared:
        assert hasattr(L, name), name


def test_format_max_and_scale(L):
    assert fpq.fpq_format_max(fpq.E4M3) == 448.0
    assert fpq.fpq_format_max(fpq.Format(4, 3, 7, fpq.SAT_PAPER)) == 480.0
    assert fpq.fpq_format_max(fpq.E2M1) == 6.0
    assert fpq.fpq_format_max(fpq.E5M2) == 57344.0
    assert fpq.fpq_format_max(fpq.Format(5, 2, 15, 0)) == 114688.0
    assert fpq.fpq_format_max(fpq.E1M2) == 1.75
    assert fpq.fpq_format_max(fpq.E3M4) == 15.5
    assert fpq.fpq_format_max(fpq.E2M5) == 3.9375
    assert fpq.fpq_format_max(fpq.Format(5, 3, 7)) == 0.0          # 9 bits
    assert fpq.fpq_format_max(fpq.Format(4, 3, 7, 5)) == 0.0        # unknown saturation mode
    # the documented range of exp_bias: 2^e - m - 104 <= exp_bias <= 126 - m
    assert fpq.fpq_format_max(fpq.Format(4, 3, 16 - 3 - 104)) == 1.875 * 2.0 ** (15 + 91)
    assert fpq.fpq_format_max(fpq.Format(4, 3, 16 - 3 - 105)) == 0.0
    assert fpq.fpq_format_max(fpq.Format(4, 3, 123)) == 1.875 * 2.0 ** (15 - 123)
    assert fpq.fpq_format_max(fpq.Format(4, 3, 124)) == 0.0
    import numpy as np
    assert fpq.fpq_scale_from_max(3.0, fpq.E4M3) == float(np.float32(3.0) / np.float32(448.0))


def test_host_side_rejections(L):
    F = fpq.E4M3.c()
    bad = fpq.Format(6, 3, 7).c()
    one = ctypes.c_void_p(16)   # never dereferenced: rejected first
    assert L.fpq_quantize_act(one, 16, 1.0, bad, one, None) == fpq.ERR_FORMAT
    assert L.fpq_quantize_act(one, -1, 1.0, F, one, None) == fpq.ERR_SHAPE
    assert L.fpq_quantize_act(None, 16, 1.0, F, one, None) == fpq.ERR_NULL
    assert L.fpq_quantize_act(one, 0, 1.0, F, one, None) == fpq.OK
    assert L.fpq_quantize_act(ctypes.c_void_p(18), 16, 1.0, F, one, None) == fpq.ERR_ALIGN
    assert L.fpq_quantize_weight(None, 4, 4, one, F, None, one, None) == fpq.ERR_NULL
    assert L.fpq_quantize_weight(one, -4, 4, one, F, None, one, None) == fpq.ERR_SHAPE
    # contraction: operand pairs
    e2m1, e3m4 = fpq.E2M1.c(), fpq.E3M4.c()
    big = ctypes.c_void_p(1024)
    # the staged forms keep to the pairs the tensor cores read
    assert L.fpq_linear_quantize_input(big, 1.0, e3m4, F, 8, 8, 8, big, 1 << 20, None) == fpq.ERR_UNSUPPORTED
    assert L.fpq_linear_quantize_input(big, 1.0, F, e3m4, 8, 8, 8, big, 1 << 20, None) == fpq.ERR_UNSUPPORTED
    paper_sat = fpq.Format(4, 3, 7, fpq.SAT_PAPER).c()
    assert L.fpq_linear_quantize_input(big, 1.0, paper_sat, F, 8, 8, 8, big, 1 << 20, None) == fpq.ERR_UNSUPPORTED
    # fpq_linear / fpq_conv2d take every valid pair (the others on the CUDA cores) and check it like any other
    assert L.fpq_linear(None, big, big, 1.0, e3m4, F, None, big, 8, 8, 8, big, 1 << 20, None) == fpq.ERR_NULL
    assert L.fpq_linear(big, big, big, 1.0, F, e3m4, None, big, 8, 8, 8, big, 8, None) == fpq.ERR_WORKSPACE
    assert L.fpq_linear(big, big, big, 1.0, F, e3m4, None, big, 8, 8, 8, ctypes.c_void_p(1032), 1 << 20, None) == fpq.ERR_ALIGN
    assert L.fpq_linear(big, big, big, 1.0, e3m4, F, None, big, 8, 8, 8, ctypes.c_void_p(1152), 1 << 20, None) == fpq.ERR_ALIGN
    assert L.fpq_linear(big, big, big, 1.0, fpq.Format(6, 3, 7).c(), F, None, big, 8, 8, 8, big, 1 << 20, None) == fpq.ERR_FORMAT
    assert L.fpq_conv2d(big, big, big, 1.0, F, e3m4, None, big, 1, 8, 2, 2, 8, 3, 3, 0, 1, big, 1 << 20, None) == fpq.ERR_SHAPE
    assert L.fpq_conv2d(big, big, big, 1.0, F, e3m4, None, big, 1, 8, 4, 4, 8, 3, 3, 1, 1, big, 16, None) == fpq.ERR_WORKSPACE
    assert L.fpq_linear(big, big, big, 1.0, F, e2m1, None, big, -1, 8, 8, big, 1 << 20, None) == fpq.ERR_SHAPE
    assert L.fpq_linear(None, big, big, 1.0, F, F, None, big, 8, 8, 8, big, 1 << 20, None) == fpq.ERR_NULL
    assert L.fpq_linear(ctypes.c_void_p(1028), big, big, 1.0, F, F, None, big, 8, 8, 8, big, 1 << 20, None) == fpq.ERR_ALIGN
    assert L.fpq_linear(big, big, big, 1.0, F, F, None, big, 8, 8, 8, big, 8, None) == fpq.ERR_WORKSPACE
    assert L.fpq_linear(big, big, big, 1.0, F, F, None, big, 8, 8, 8, None, 0, None) == fpq.ERR_WORKSPACE
    assert L.fpq_linear(big, big, big, 1.0, F, F, None, big, 0, 8, 8, None, 0, None) == fpq.OK
    assert L.fpq_conv2d(big, big, big, 1.0, F, F, None, big, 1, 8, 2, 2, 8, 3, 3, 0, 1, big, 1 << 20, None) == fpq.ERR_SHAPE
    assert L.fpq_conv2d(big, big, big, 1.0, F, F, None, big, 1, 8, 4, 4, 8, 3, 3, 1, 0, big, 1 << 20, None) == fpq.ERR_SHAPE
    assert L.fpq_conv2d(big, big, big, 1.0, F, F, None, big, 1, 8, 4, 4, 8, 3, 3, 1, 1, big, 16, None) == fpq.ERR_WORKSPACE


def test_search_host_side(L):
    import numpy as np
    import oracle as O
    enc = (fpq._CFormat * 2)(fpq.Format(1, 2, 1).c(), fpq.Format(2, 1, 2).c())
    encp = ctypes.cast(enc, ctypes.c_void_p)
    big = ctypes.c_void_p(1024)
    assert L.fpq_search_format(big, -1, encp, 2, big, 4, big, big, big, 1 << 30, None) == fpq.ERR_SHAPE
    assert L.fpq_search_format(big, 8, encp, 0, big, 4, big, big, big, 1 << 30, None) == fpq.ERR_SHAPE
    assert L.fpq_search_format(big, 8, encp, 2, big, 257, big, big, big, 1 << 30, None) == fpq.ERR_SHAPE
    assert L.fpq_search_format(None, 8, encp, 2, big, 4, big, big, big, 1 << 30, None) == fpq.ERR_NULL
    assert L.fpq_search_format(big, 8, encp, 2, big, 4, ctypes.c_void_p(1028), big, big, 1 << 30, None) == fpq.ERR_ALIGN
    assert L.fpq_search_format(big, 8, encp, 2, big, 4, big, big, big, 64, None) == fpq.ERR_WORKSPACE
    native = (fpq._CFormat * 1)(fpq.E4M3.c())
    assert L.fpq_search_format(big, 8, ctypes.cast(native, ctypes.c_void_p), 1, big, 4, big, big, big, 1 << 30,
                               None) == fpq.ERR_UNSUPPORTED
    assert fpq.fpq_search_workspace_size(4, 111) == 1184 * 444 * 8
    assert fpq.fpq_search_workspace_size(8, 256) == 0            # more than 1024 candidates
    # the clipping candidates are the oracle's, bit for bit
    for maxabs in (3.7, 0.0123, 1e4):
        assert np.array_equal(fpq.fpq_search_clip_candidates(maxabs, 111).numpy(), O.clip_candidates(maxabs, 111))
    assert L.fpq_search_clip_candidates(0.0, 5, big) == fpq.ERR_SHAPE
    assert L.fpq_search_clip_candidates(1.0, 0, big) == fpq.ERR_SHAPE
    assert L.fpq_search_clip_candidates(float("inf"), 5, big) == fpq.ERR_SHAPE


def test_sizes(L):
    assert fpq.fpq_linear_workspace_size(100, 64, 320, fpq.E4M3, fpq.E4M3) == 100 * 320
    assert fpq.fpq_linear_workspace_size(100, 64, 321, fpq.E4M3, fpq.E2M1) == 100 * 336
    # E3M4 activations as two E4M3 terms: codes [100][2 * 384], then the weights' rows repeated [64][2 * 384]
    assert fpq.fpq_linear_workspace_size(100, 64, 320, fpq.E3M4, fpq.E4M3) == 100 * 768 + 64 * 768
    assert fpq.fpq_linear_workspace_size(100, 64, 320, fpq.E3M4, fpq.E2M1) == 100 * 768 + 64 * 384      # packed FP4 weights
    # a 6-bit format inside E4M3: one term, no copy of the weights
    assert fpq.fpq_linear_workspace_size(100, 64, 320, fpq.Format(3, 2, 3), fpq.E4M3) == 100 * 384
    # term activations against two-term weights, or activations beyond two terms: FP32 scratch of the grid-value route
    assert fpq.fpq_linear_workspace_size(100, 64, 320, fpq.E3M4, fpq.E3M4) > 4 * 100 * 320
    assert fpq.fpq_linear_workspace_size(100, 64, 320, fpq.Format(6, 1, 31), fpq.E4M3) > 4 * 100 * 320
    assert fpq.fpq_conv2d_workspace_size(2, 4, 8, 8, 16, 3, 3, 1, 1, fpq.E2M5, fpq.E4M3) == 2 * 100 * 256 + 16 * 9 * 256
    assert fpq.fpq_linear_workspace_size(100, 64, 320, fpq.E5M2, fpq.E2M1) == 100 * 320    # OCP E5M2 activations: tensor cores
    assert fpq.fpq_linear_workspace_size(100, 64, 320, fpq.Format(6, 3, 7), fpq.E4M3) == 0
    assert fpq.fpq_conv2d_workspace_size(2, 4, 8, 8, 16, 3, 3, 1, 1, fpq.E4M3, fpq.E2M1) == 2 * 100 * 16
    assert fpq.fpq_prepared_size(fpq.E4M3, fpq.LINEAR, 10, 320) == 10 * 384
    assert fpq.fpq_prepared_size(fpq.E2M1, fpq.CONV2D, 10, 320, 3, 3) == 10 * 9 * 384 // 2
    assert fpq.fpq_prepared_size(fpq.E2M1, fpq.LINEAR, 10, 320, 3, 3) == 0
    assert fpq.status_string(fpq.ERR_TIMEOUT) == "device-side wait timed out"


def test_round_learn_rejections(L):
    p = ctypes.c_void_p(256)   # never dereferenced: rejected first
    F = fpq.E2M1.c()
    assert L.fpq_round_learn_step(p, p, fpq.Format(6, 3, 7).c(), p, p, 4, 4, 4, 0.0, 0.0, p, p, p, 1 << 30, None) == fpq.ERR_FORMAT
    assert L.fpq_round_learn_step(p, p, F, p, p, 0, 4, 4, 0.0, 0.0, p, p, p, 1 << 30, None) == fpq.ERR_SHAPE
    assert L.fpq_round_learn_step(p, p, F, None, p, 4, 4, 4, 0.0, 0.0, p, p, p, 1 << 30, None) == fpq.ERR_NULL
    assert L.fpq_round_learn_step(p, p, F, p, p, 4, 4, 4, 0.0, 0.0, p, ctypes.c_void_p(260), p, 1 << 30, None) == fpq.ERR_ALIGN
    assert L.fpq_round_learn_step(p, p, F, p, p, 4, 4, 4, 0.0, 0.0, p, p, p, 16, None) == fpq.ERR_WORKSPACE
    assert L.fpq_round_learn_step(p, p, F, p, p, 4, 4, 4, float("nan"), 0.0, p, p, p, 1 << 30, None) == fpq.ERR_SHAPE
    assert L.fpq_round_learn_workspace_size(0, 4, 4) == 0


def test_weight_formats_the_layer_accepts(L):
    F = fpq.E4M3.c()
    big = ctypes.c_void_p(1024)

    def accepted(fw):
        # (by the tensor-core forms) a NULL activation pointer is rejected after the operand pair has been checked
        return L.fpq_linear_quantize_input(None, 1.0, F, fw.c(), 8, 8, 8, big, 1 << 20, None) != fpq.ERR_UNSUPPORTED

    # read by the tensor cores as they are (E4M3, E2M1 and the OCP E5M2)
    assert accepted(fpq.E4M3) and accepted(fpq.E2M1) and accepted(fpq.E5M2)
    # every value is also an E4M3 value: re-encoded when the weights are prepared
    assert accepted(fpq.E1M2) and accepted(fpq.Format(2, 1, 2)) and accepted(fpq.Format(3, 2, 3))
    # more mantissa bits or a wider exponent range than E4M3 holds, or the code 480 of the paper's E4M3
    assert not accepted(fpq.E3M4) and not accepted(fpq.E2M5) and not accepted(fpq.Format(5, 2, 16, fpq.SAT_PAPER))
    assert not accepted(fpq.Format(4, 3, 7, fpq.SAT_PAPER)) and not accepted(fpq.Format(4, 3, 8, fpq.SAT_NATIVE))
    # E3M4 / E2M5 weights are prepared as two E4M3 terms: twice the bytes, twice the activation codes
    d = fpq._CLayerDesc(fpq.LINEAR, 8, 200, 1, 1)
    assert L.fpq_prepared_size(fpq.E3M4.c(), ctypes.byref(d)) == 2 * 8 * 256
    assert L.fpq_prepared_size(fpq.E5M2.c(), ctypes.byref(d)) == 8 * 256       # read as it is
    # the paper's default E4M3 (bias 8): two terms after a factor of two that the dequantization scale takes back
    assert L.fpq_prepared_size(fpq.Format(4, 3, 8, fpq.SAT_PAPER).c(), ctypes.byref(d)) == 2 * 8 * 256
    # the paper's E5M2 (bias 16, all exponent fields finite): two terms of the tensor cores' own E5M2
    assert L.fpq_prepared_size(fpq.Format(5, 2, 16, fpq.SAT_PAPER).c(), ctypes.byref(d)) == 2 * 8 * 256
    # 7 significant bits are 4 + 3: two terms again
    assert L.fpq_prepared_size(fpq.Format(1, 6, 1, fpq.SAT_PAPER).c(), ctypes.byref(d)) == 2 * 8 * 256
    # 64 binades fit no two terms of a tensor-core type: CUDA cores, codes as they are
    assert L.fpq_prepared_size(fpq.Format(6, 1, 31, fpq.SAT_PAPER).c(), ctypes.byref(d)) == 8 * 256
    assert fpq.fpq_linear_workspace_size(100, 64, 200, fpq.E4M3, fpq.E2M5) == 100 * 512
    assert L.fpq_prepared_size(fpq.E2M1.c(), ctypes.byref(d)) == 8 * 256 // 2
    assert L.fpq_prepared_size(fpq.E1M2.c(), ctypes.byref(d)) == 8 * 256      # one E4M3 byte per weight
    assert L.fpq_prepared_size(fpq.E4M3.c(), ctypes.byref(d)) == 8 * 256


def test_activation_scales_are_checked_before_anything_else(L):
    F = fpq.E4M3.c()
    p = ctypes.c_void_p(1024)      # never dereferenced
    for bad in (0.0, -1.0, float("inf"), float("nan")):
        assert L.fpq_quantize_act(p, 16, bad, F, p, None) == fpq.ERR_SCALE
        assert L.fpq_linear(p, p, p, bad, F, F, None, p, 8, 8, 8, p, 1 << 20, None) == fpq.ERR_SCALE
        assert L.fpq_conv2d(p, p, p, bad, F, F, None, p, 1, 4, 4, 4, 4, 3, 3, 1, 1, p, 1 << 20, None) == fpq.ERR_SCALE
        assert L.fpq_linear_quantize_input(p, bad, F, F, 8, 8, 8, p, 1 << 20, None) == fpq.ERR_SCALE
        assert L.fpq_conv2d_split(p, 4, bad, p, 4, 1.0, p, p, F, F, None, p, 1, 4, 4, 4, 3, 3, 1, 1, p, 1 << 20, None) == fpq.ERR_SCALE
        assert L.fpq_conv2d_split(p, 4, 1.0, p, 4, bad, p, p, F, F, None, p, 1, 4, 4, 4, 3, 3, 1, 1, p, 1 << 20, None) == fpq.ERR_SCALE
    assert "scale" in fpq.status_string(fpq.ERR_SCALE)


def test_route_query(L):
    try:
        # the workload the bench times: one 128-channel chunk, 128 outputs -> the CTA-pair kernel
        assert fpq.fpq_conv2d_route(64, 128, 32, 32, 128, 3, 3, 1, 1, fpq.E4M3, fpq.E4M3) == fpq.ROUTE_PAIR_FUSED
        # weights that do not fit the shared memory of two SMs, more than 256 outputs, a stride: two kernels
        assert fpq.fpq_conv2d_route(2, 1280, 16, 16, 1280, 3, 3, 1, 1, fpq.E4M3, fpq.E2M1) == fpq.ROUTE_TWO_KERNELS
        assert fpq.fpq_conv2d_route(2, 128, 32, 32, 512, 1, 1, 0, 1, fpq.E4M3, fpq.E4M3) == fpq.ROUTE_TWO_KERNELS
        assert fpq.fpq_conv2d_route(2, 128, 32, 32, 128, 3, 3, 1, 2, fpq.E4M3, fpq.E4M3) == fpq.ROUTE_TWO_KERNELS
        # formats without a tensor-core type
        assert fpq.fpq_conv2d_route(2, 128, 32, 32, 128, 3, 3, 1, 1, fpq.E3M4, fpq.E4M3) == fpq.ROUTE_OTHER
        assert L.fpq_conv2d_route(2, 128, 32, 32, 128, 3, 3, 1, 1, fpq.Format(6, 3, 7).c(), fpq.E4M3.c()) == fpq.ERR_FORMAT
        assert L.fpq_conv2d_route(2, 0, 32, 32, 128, 3, 3, 1, 1, fpq.E4M3.c(), fpq.E4M3.c()) == fpq.ERR_SHAPE
        fpq.fpq_set_path_policy(fpq.PATH_TWO_KERNELS)
        assert fpq.fpq_conv2d_route(64, 128, 32, 32, 128, 3, 3, 1, 1, fpq.E4M3, fpq.E4M3) == fpq.ROUTE_TWO_KERNELS
        fpq.fpq_set_path_policy(fpq.PATH_FUSED)
        assert fpq.fpq_conv2d_route(2, 1280, 16, 16, 1280, 3, 3, 1, 1, fpq.E4M3, fpq.E2M1) == fpq.ROUTE_FUSED
    finally:
        fpq.fpq_set_path_policy(fpq.PATH_AUTO)
    assert L.fpq_selftest_bounded_wait(0, None) == fpq.ERR_SHAPE
    assert L.fpq_selftest_bounded_wait(1 << 40, None) == fpq.ERR_SHAPE
