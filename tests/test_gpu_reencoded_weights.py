"""Layers whose weights are in an encoding the tensor cores do not read directly (E1M2, the FP4
alternative the encoding search of Sec. V-A may select; E2M1 with the paper's default bias 2; small
6-bit formats): the weight codes are re-encoded exactly into E4M3 when the weights are prepared, so the
results must meet the same bar as the native formats."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2408_06995_b200 as fpq
from paper_2408_06995_b200 import inputs as I
from _helpers import FMT, assert_close, gpu_layer, layer_scales, oracle_layer

pytestmark = pytest.mark.gpu

REENCODED = ["e1m2", "e2m1b2", "e3m2b3", "e2m3b1"]


def _check_full(L, use_bias=True):
    ws, xs = layer_scales(L)
    y = gpu_layer(L, ws, xs, use_bias)
    yr, ab = oracle_layer(L, ws, xs, None, use_bias)
    assert y.shape == yr.shape
    return assert_close(y, yr, ab)


@pytest.mark.parametrize("wfmt", REENCODED)
@pytest.mark.parametrize("M,K,N", [(130, 200, 72), (300, 320, 960), (2, 1280, 320), (257, 1000, 4)])
def test_linear(wfmt, M, K, N):
    L = I.linear_layer("t", M, K, N, wfmt, rounding=(FMT[wfmt][1].bits == 4))
    I.draw(L, 21, M + K + N, "normal", 0.02, True, 0.01, (0.001, 20.0))
    _check_full(L)


@pytest.mark.parametrize("wfmt", ["e1m2", "e3m2b3"])
@pytest.mark.parametrize("shape", [(2, 40, 12, 12, 72, 3, 1), (1, 130, 9, 11, 33, 3, 2), (3, 64, 8, 8, 130, 1, 1)])
def test_conv(wfmt, shape):
    B, C, H, W, Co, R, stride = shape
    L = I.conv_layer("t", B, C, H, W, Co, R, stride=stride, wfmt=wfmt, rounding=(FMT[wfmt][1].bits == 4))
    I.draw(L, 22, B + C + Co, "silu", 0.03, True, 0.01)
    _check_full(L)


def test_prepared_copy_holds_the_same_values_in_e4m3():
    # every E1M2 code, through the encoder and the prepared copy: decoded as E4M3 it is the same number
    f_g, f_o = FMT["e1m2"]
    table = O.decode_table(f_o)
    vals = np.unique(table)
    K = 128
    w = np.resize(vals, (4, K)).astype(np.float32)
    scale = np.ones(4, dtype=np.float32)
    codes = fpq.fpq_quantize_weight(torch.from_numpy(w).cuda(), torch.from_numpy(scale).cuda(), f_g, None)
    prep = fpq.fpq_prepare_weight(codes, f_g, fpq.LINEAR, 4, K)
    assert prep.numel() == 4 * K                              # one byte per weight
    back = prep.view(torch.float8_e4m3fn).to(torch.float32).cpu().numpy().reshape(4, K)
    assert np.array_equal(back, w)


def test_search_result_runs_as_a_layer():
    # the FP4 search picks one of (E1M2, E2M1 with bias 2); either choice must be usable by the layer
    rng = np.random.default_rng(3)
    M, K, N = 96, 256, 64
    x = rng.standard_normal((M, K)).astype(np.float32)
    w = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    for i, enc in enumerate(O.FP4_ENCODINGS):
        g = fpq.Format(enc.e, enc.m, enc.B, fpq.SAT_PAPER)
        L = I.linear_layer("t", M, K, N, "e1m2" if enc.e == 1 else "e2m1b2")
        L.x, L.w, L.bias, L.bits = x, w, np.zeros(N, np.float32), None
        assert FMT[L.wfmt][0].c().exp_bits == g.c().exp_bits and FMT[L.wfmt][0].c().exp_bias == g.c().exp_bias
        _check_full(L, use_bias=False)


# OCP E5M2 (bias 15, native saturation) is the tensor cores' second 8-bit operand type: read as it is
@pytest.mark.parametrize("M,K,N", [(130, 200, 72), (300, 320, 960), (2, 1280, 320), (257, 1000, 4)])
def test_linear_e5m2_native_weights(M, K, N):
    L = I.linear_layer("t", M, K, N, "e5m2", rounding=True)
    I.draw(L, 23, M + K + N, "normal", 0.02, True, 0.01, (0.001, 20.0))
    _check_full(L)


@pytest.mark.parametrize("shape", [(2, 40, 12, 12, 72, 3, 1), (1, 130, 9, 11, 33, 3, 2), (2, 256, 8, 8, 256, 3, 1)])
def test_conv_e5m2_native_weights(shape):
    B, C, H, W, Co, R, stride = shape
    L = I.conv_layer("t", B, C, H, W, Co, R, stride=stride, wfmt="e5m2", rounding=True)
    I.draw(L, 24, B + C + Co, "silu", 0.03, True, 0.01)
    _check_full(L)
