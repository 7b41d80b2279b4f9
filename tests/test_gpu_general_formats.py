"""Layers whose operand formats the tensor cores have no type for (E3M4, E2M5, E5M2, the paper's E4M3 with
all exponent fields finite - what the FP8 encoding search of Sec. V-A may select - or activations in a format
other than native E4M3): fpq_linear / fpq_conv2d run them as terms of a tensor-core type where the format splits
into one or two, else on FP32 grid values, always with the same arithmetic model (exact products of grid values, FP32
sums), so the bar is the one of the native path."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2408_06995_b200 as fpq
from paper_2408_06995_b200 import inputs as I
from _helpers import assert_close, to_oracle

pytestmark = pytest.mark.gpu

E4M3_PAPER = fpq.Format(4, 3, 7, fpq.SAT_PAPER)
E4M3_B8 = fpq.Format(4, 3, 8, fpq.SAT_PAPER)        # the paper's default bias 2^(e-1)
E5M2_B16 = fpq.Format(5, 2, 16, fpq.SAT_PAPER)
E2M1_TINY = fpq.Format(2, 1, 12, fpq.SAT_PAPER)      # a 4-bit format whose values E4M3 cannot hold as they are
E1M6 = fpq.Format(1, 6, 1, fpq.SAT_PAPER)            # 7 significant bits = 4 + 3: two E4M3 terms
E6M1 = fpq.Format(6, 1, 31, fpq.SAT_PAPER)           # 64 binades: beyond any two tensor-core terms, CUDA cores
E5M2_B40 = fpq.Format(5, 2, 40, fpq.SAT_PAPER)       # needs a factor beyond the 2^16 the split tries
E3M2_B3 = fpq.Format(3, 2, 3, fpq.SAT_PAPER)         # 6-bit formats whose every value is an E4M3 value: one term
E2M3_B1 = fpq.Format(2, 3, 1, fpq.SAT_PAPER)

PAIRS = [(fpq.E4M3, fpq.E3M4), (fpq.E4M3, fpq.E2M5), (fpq.E4M3, fpq.E5M2), (fpq.E4M3, E5M2_B16), (fpq.E4M3, E4M3_PAPER),
         (fpq.E4M3, E4M3_B8), (fpq.E4M3, E2M1_TINY), (fpq.E4M3, E1M6), (fpq.E4M3, E6M1), (fpq.E4M3, E5M2_B40), (fpq.E3M4, E5M2_B16),
         (fpq.E5M2, fpq.E4M3), (fpq.E3M4, fpq.E2M1), (E4M3_PAPER, fpq.E1M2), (fpq.E2M5, fpq.E3M4),
         # OCP E5M2 activations are read by the tensor cores as they are, with every kind of weight preparation
         (fpq.E5M2, fpq.E5M2), (fpq.E5M2, fpq.E2M1), (fpq.E5M2, fpq.E1M2), (fpq.E5M2, fpq.E3M4), (fpq.E5M2, E5M2_B16),
         # activations that are one or two terms of a tensor-core type, against weights read as they are or re-encoded:
         # the terms are written as operand codes and the ordinary contraction runs over them
         (fpq.E3M4, fpq.E4M3), (fpq.E2M5, fpq.E4M3), (fpq.E2M5, fpq.E2M1), (fpq.E2M5, fpq.E5M2), (E4M3_PAPER, fpq.E4M3),
         (E4M3_B8, fpq.E4M3), (E5M2_B16, fpq.E2M1), (E3M2_B3, fpq.E4M3), (E2M3_B1, fpq.E2M1), (E1M6, fpq.E1M2)]


def _run(L, gfx, gfw, use_bias=True):
    ofx, ofw = to_oracle(gfx), to_oracle(gfw)
    d = "cuda"
    w2 = L.w.reshape(L.N, -1)
    ws = np.array([fpq.fpq_scale_from_max(float(v), gfw) for v in np.abs(w2).max(axis=1)], dtype=np.float32)
    assert np.array_equal(ws, np.array([O.scale_from_max(v, ofw) for v in np.abs(w2).max(axis=1)], dtype=np.float32))
    xs = fpq.fpq_scale_from_max(float(np.abs(L.x).max()), gfx)
    assert np.float32(xs) == O.scale_from_max(float(np.abs(L.x).max()), ofx)
    rb = O.pack_bits(L.bits) if L.bits is not None else None
    codes = fpq.fpq_quantize_weight(torch.from_numpy(w2).to(d), torch.from_numpy(ws).to(d), gfw,
                                    None if rb is None else torch.from_numpy(rb).to(d))
    assert np.array_equal(codes.cpu().numpy(), O.quantize_weight(w2, ws, ofw, rb))
    x = torch.from_numpy(L.x).to(d)
    bias = torch.from_numpy(L.bias).to(d) if use_bias else None
    wsd = torch.from_numpy(ws).to(d)
    if L.kind == "linear":
        prep = fpq.fpq_prepare_weight(codes, gfw, fpq.LINEAR, L.N, L.K)
        y = fpq.fpq_linear(x, prep, wsd, xs, gfx, gfw, bias, L.N)
        yr, ab = O.linear(L.x, L.w, ws, xs, ofx, ofw, L.bias if use_bias else None, rb)
    else:
        prep = fpq.fpq_prepare_weight(codes, gfw, fpq.CONV2D, L.N, L.C, L.R, L.S)
        y = fpq.fpq_conv2d(x, prep, wsd, xs, gfx, gfw, bias, L.N, L.R, L.S, L.pad, L.stride)
        yr, ab = O.conv2d(L.x, L.w, ws, xs, ofx, ofw, L.bias if use_bias else None, rb, L.pad, L.stride)
    assert fpq.fpq_read_status() == fpq.OK
    y = y.cpu().numpy()
    assert y.shape == yr.shape
    return assert_close(y, yr, ab)


@pytest.mark.parametrize("gfx,gfw", PAIRS)
@pytest.mark.parametrize("M,K,N", [(130, 200, 72), (300, 320, 260), (2, 129, 5)])
def test_linear(gfx, gfw, M, K, N):
    L = I.linear_layer("t", M, K, N, rounding=(M == 130))
    I.draw(L, 31, M + K + N, "normal", 0.02, True, 0.01, (0.001, 20.0))
    _run(L, gfx, gfw)
    _run(L, gfx, gfw, use_bias=False)


@pytest.mark.parametrize("gfx,gfw", [(fpq.E4M3, fpq.E3M4), (fpq.E4M3, E5M2_B16), (fpq.E4M3, E4M3_B8), (fpq.E5M2, fpq.E2M1),
                                     (fpq.E3M4, fpq.E1M2), (fpq.E5M2, fpq.E4M3), (fpq.E5M2, fpq.E3M4),
                                     (fpq.E2M5, fpq.E4M3), (fpq.E3M4, fpq.E2M1), (E3M2_B3, fpq.E4M3), (E5M2_B16, fpq.E4M3)])
@pytest.mark.parametrize("shape", [(2, 40, 12, 12, 72, 3, 1), (1, 130, 9, 11, 33, 3, 2), (3, 64, 8, 8, 130, 1, 1)])
def test_conv(gfx, gfw, shape):
    B, C, H, W, Co, R, stride = shape
    L = I.conv_layer("t", B, C, H, W, Co, R, stride=stride, rounding=(stride == 2))
    I.draw(L, 32, B + C + Co, "silu", 0.03, True, 0.01)
    _run(L, gfx, gfw)


def test_e5m2_activations_at_a_size_that_spans_many_tiles():
    # the tensor-core route for OCP E5M2 activations on shapes with several tiles per CTA and a ragged tail
    L = I.linear_layer("t", 1000, 320, 960, "e4m3")
    I.draw(L, 35, 1, "normal", 0.02, True, 0.01, (0.001, 20.0))
    _run(L, fpq.E5M2, fpq.E4M3)
    L = I.conv_layer("t", 9, 256, 32, 32, 256, 3, wfmt="e2m1", rounding=True)      # wide-MMA contraction (CTA pairs)
    I.draw(L, 35, 2, "silu", 0.03, True, 0.01)
    _run(L, fpq.E5M2, fpq.E2M1)
    # the scratch is one byte per activation: the tensor-core route, not the FP32 scratch of the CUDA-core route
    assert fpq.fpq_linear_workspace_size(1000, 960, 320, fpq.E5M2, fpq.E4M3) == 1000 * 320
    assert fpq.fpq_linear_workspace_size(1000, 960, 320, fpq.E3M4, fpq.E4M3) > 4 * 1000 * 320


@pytest.mark.parametrize("gfx", [fpq.E3M4, fpq.E2M5])
def test_two_term_activations_at_a_size_that_spans_many_tiles(gfx):
    # the FP8 activation encodings of the search that the tensor cores have no type for, as two E4M3 terms:
    # several tiles per CTA, a ragged tail, both weight widths; and a convolution with a split reduction
    L = I.linear_layer("t", 1000, 320, 960, "e4m3")
    I.draw(L, 36, 1, "normal", 0.02, True, 0.01, (0.001, 20.0))
    _run(L, gfx, fpq.E4M3)
    _run(L, gfx, fpq.E2M1)
    L = I.conv_layer("t", 2, 320, 16, 16, 320, 3)
    I.draw(L, 36, 2, "silu", 0.03, True, 0.01)
    _run(L, gfx, fpq.E2M1)


def test_four_bit_activation_format_as_one_term():
    # E1M2 activations (every value an E4M3 value): the oracle's layer reads 4-bit activation codes packed per row,
    # which equals the flat packing of its quantizer for even row lengths only
    L = I.linear_layer("t", 130, 200, 72)
    I.draw(L, 37, 1, "normal", 0.02, True, 0.01, (0.001, 20.0))
    _run(L, fpq.E1M2, fpq.E4M3)
    _run(L, fpq.E1M2, fpq.E2M1)


def test_every_fp8_search_candidate_runs_as_a_layer():
    # the four FP8 encodings of Algorithm 1 with the paper's default bias, as weight formats of one layer
    L = I.linear_layer("t", 96, 256, 64)
    I.draw(L, 33, 0, "normal", 0.02, True, 0.01)
    for enc in O.FP8_ENCODINGS:
        _run(L, fpq.E4M3, fpq.Format(enc.e, enc.m, enc.B, fpq.SAT_PAPER))


@pytest.mark.parametrize("gfw", [fpq.E3M4, E5M2_B16])
def test_empty_and_nan_inputs(gfw):
    d = "cuda"
    N, K = 8, 32
    w = torch.randn((N, K), device=d) * 0.02
    ws = (w.abs().amax(dim=1) / fpq.fpq_format_max(gfw)).contiguous()
    prep = fpq.fpq_prepare_weight(fpq.fpq_quantize_weight(w, ws, gfw, None), gfw, fpq.LINEAR, N, K)
    # no rows: nothing to do, no error
    y0 = fpq.fpq_linear(torch.empty((0, K), device=d), prep, ws, 0.01, fpq.E4M3, gfw, None, N)
    assert y0.shape == (0, N) and fpq.fpq_read_status() == fpq.OK
    # a NaN activation is quantized to zero and reported through the status word
    x = torch.randn((16, K), device=d)
    x[3, 5] = float("nan")
    y = fpq.fpq_linear(x, prep, ws, 0.01, fpq.E4M3, gfw, None, N)
    assert fpq.fpq_read_status() == fpq.ERR_NAN_INPUT
    assert torch.isfinite(y).all()
    x[3, 5] = 0.0
    y2 = fpq.fpq_linear(x, prep, ws, 0.01, fpq.E4M3, gfw, None, N)
    assert fpq.fpq_read_status() == fpq.OK
    assert torch.equal(y, y2)


@pytest.mark.parametrize("bits", [8, 4])
def test_search_choice_for_the_weights_runs_as_the_layer(bits):
    # Sec. V-A end to end: Algorithm 1 picks an encoding and a clipping value for the weight tensor (per tensor, as
    # in the paper), the clipping value becomes the scale, and the layer runs with exactly that format
    L = I.linear_layer("t", 160, 384, 96)
    I.draw(L, 34, bits, "normal", 0.02, False, 0.01)
    encs_o = O.FP8_ENCODINGS if bits == 8 else O.FP4_ENCODINGS
    encs_g = [fpq.Format(f.e, f.m, f.B, fpq.SAT_PAPER) for f in encs_o]
    clips = fpq.fpq_search_clip_candidates(float(np.abs(L.w).max()), 111)
    _, best = fpq.fpq_search_format(torch.from_numpy(L.w.reshape(-1)).cuda(), encs_g, clips.cuda())
    i, j = (int(v) for v in best.cpu().numpy())
    gfw, ofw = encs_g[i], encs_o[i]
    scale = np.float32(clips.numpy()[j]) / np.float32(O.cmax(ofw))          # c = scale * c(F)
    ws = np.full(L.N, scale, dtype=np.float32)
    xs = fpq.fpq_scale_from_max(float(np.abs(L.x).max()), fpq.E4M3)
    d = "cuda"
    codes = fpq.fpq_quantize_weight(torch.from_numpy(L.w).to(d), torch.from_numpy(ws).to(d), gfw, None)
    assert np.array_equal(codes.cpu().numpy(), O.quantize_weight(L.w, ws, ofw, None))
    prep = fpq.fpq_prepare_weight(codes, gfw, fpq.LINEAR, L.N, L.K)
    y = fpq.fpq_linear(torch.from_numpy(L.x).to(d), prep, torch.from_numpy(ws).to(d), xs, fpq.E4M3, gfw,
                       torch.from_numpy(L.bias).to(d), L.N)
    assert fpq.fpq_read_status() == fpq.OK
    yr, ab = O.linear(L.x, L.w, ws, xs, O.E4M3, ofw, L.bias, None)
    assert_close(y.cpu().numpy(), yr, ab)
