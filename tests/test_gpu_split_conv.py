"""Convolution over two concatenated inputs quantized with their own scales (Sec. VI-A) against the
oracle.  The oracle has no routine of its own for this layer: by linearity it is the sum of two
ordinary quantized convolutions, one per input tensor, over the matching slices of the weights."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2408_06995_b200 as fpq
from _helpers import FMT, assert_close, Guarded

pytestmark = pytest.mark.gpu


def _draw(B, C1, C2, H, W, Co, R, seed, spread):
    rng = np.random.default_rng(seed)
    z = rng.standard_normal((B, C1, H, W))
    x1 = (z / (1 + np.exp(-z))).astype(np.float32)                      # previous layer's output
    x2 = (rng.standard_normal((B, C2, H, W)) * spread).astype(np.float32)   # skip connection, wider
    w = (rng.standard_normal((Co, C1 + C2, R, R)) * 0.03 * rng.uniform(0.5, 2, (Co, 1, 1, 1))).astype(np.float32)
    bias = (rng.standard_normal(Co) * 0.01).astype(np.float32)
    bits = rng.integers(0, 2, (Co, (C1 + C2) * R * R)).astype(np.uint8)
    return x1, x2, w, bias, bits


def _oracle(x1, x2, w, bias, bits, ws, s1, s2, ofw, pad, stride):
    Co, C, R, S = w.shape
    C1 = x1.shape[1]
    b3 = bits.reshape(Co, C, R * S)
    ya, aa = O.conv2d(x1, w[:, :C1], ws, s1, O.E4M3, ofw, bias, O.pack_bits(b3[:, :C1].reshape(Co, -1)), pad, stride)
    yb, ab = O.conv2d(x2, w[:, C1:], ws, s2, O.E4M3, ofw, None, O.pack_bits(b3[:, C1:].reshape(Co, -1)), pad, stride)
    return ya + yb, aa + ab


def _gpu(x1, x2, w, bias, bits, ws, s1, s2, gfw, pad, stride):
    Co, C, R, S = w.shape
    B, C1, H, W = x1.shape
    C2 = x2.shape[1]
    dev = "cuda"
    codes = fpq.fpq_quantize_weight(torch.from_numpy(w.reshape(Co, -1)).to(dev), torch.from_numpy(ws).to(dev), gfw,
                                    torch.from_numpy(O.pack_bits(bits)).to(dev))
    prep = fpq.fpq_prepare_weight_split(codes, gfw, Co, C1, C2, R, S)
    Ho, Wo = (H + 2 * pad - R) // stride + 1, (W + 2 * pad - S) // stride + 1
    yg = Guarded(4 * B * Co * Ho * Wo)                                   # guard bands around output and scratch
    wg = Guarded(fpq.fpq_conv2d_split_workspace_size(B, C1, C2, H, W, Co, R, S, pad, stride, fpq.E4M3, gfw))
    y, wk = yg.f32((B, Co, Ho, Wo)), wg.inner
    wk.fill_(0xAB)                                                       # the call must not rely on a clean scratch
    fpq.fpq_conv2d_split(torch.from_numpy(x1).to(dev), s1, torch.from_numpy(x2).to(dev), s2, prep,
                         torch.from_numpy(ws).to(dev), fpq.E4M3, gfw, torch.from_numpy(bias).to(dev), y, R, S, pad,
                         stride, wk)
    assert fpq.fpq_read_status() == fpq.OK
    yg.check("two-tensor convolution output")
    wg.check("two-tensor convolution workspace")
    return y.cpu().numpy()


def _scales(x1, x2, w, gfw):
    ws = np.array([fpq.fpq_scale_from_max(float(v), gfw) for v in np.abs(w.reshape(w.shape[0], -1)).max(axis=1)],
                  dtype=np.float32)
    return ws, fpq.fpq_scale_from_max(float(np.abs(x1).max()), fpq.E4M3), \
        fpq.fpq_scale_from_max(float(np.abs(x2).max()), fpq.E4M3)


@pytest.mark.parametrize("wfmt", ["e4m3", "e2m1"])
@pytest.mark.parametrize("B,C1,C2,H,W,Co,R,pad,stride", [
    (2, 128, 128, 8, 8, 96, 3, 1, 1),       # both tensors one chunk
    (2, 320, 320, 8, 8, 200, 3, 1, 1),      # SD-like 640 = 320 + 320: the boundary is not a multiple of 128
    (1, 640, 320, 8, 8, 130, 3, 1, 1),      # unequal tensors, several CTAs each
    (2, 20, 7, 9, 7, 37, 3, 1, 1),          # tiny ragged channels
    (2, 200, 72, 16, 16, 64, 1, 0, 1),      # 1x1 skip convolution, 64-column tiles
    (2, 130, 140, 16, 16, 24, 3, 1, 2),     # stride 2
    (8, 64, 64, 32, 32, 140, 3, 1, 1),      # many tiles: one pair of CTAs per tile
])
def test_split_conv_matches_the_sum_of_two_oracle_convolutions(wfmt, B, C1, C2, H, W, Co, R, pad, stride):
    gfw, ofw = FMT[wfmt]
    x1, x2, w, bias, bits = _draw(B, C1, C2, H, W, Co, R, B + C1 + C2 + Co, 3.0)
    ws, s1, s2 = _scales(x1, x2, w, gfw)
    assert s1 != s2
    got = _gpu(x1, x2, w, bias, bits, ws, s1, s2, gfw, pad, stride)
    want, ab = _oracle(x1, x2, w, bias, bits, ws, s1, s2, ofw, pad, stride)
    assert_close(got, want, ab)
    # twice in a row on the same scratch gives the same bits
    assert np.array_equal(got, _gpu(x1, x2, w, bias, bits, ws, s1, s2, gfw, pad, stride))


def test_equal_scales_reduce_to_the_ordinary_convolution_of_the_concatenation():
    gfw, ofw = FMT["e4m3"]
    x1, x2, w, bias, bits = _draw(2, 96, 160, 8, 8, 72, 3, 5, 1.0)
    ws, s1, s2 = _scales(x1, x2, w, gfw)
    s = max(s1, s2)
    got = _gpu(x1, x2, w, bias, bits, ws, s, s, gfw, 1, 1)
    want, ab = O.conv2d(np.concatenate([x1, x2], axis=1), w, ws, s, O.E4M3, ofw, bias, O.pack_bits(bits), 1, 1)
    assert_close(got, want, ab)


def test_split_sizes_and_rejections():
    assert fpq.lib().fpq_prepared_size_split(fpq.E4M3.c(), 10, 320, 320, 3, 3) == 10 * 9 * (384 + 384)
    assert fpq.lib().fpq_prepared_size_split(fpq.E2M1.c(), 10, 100, 7, 1, 1) == 10 * (128 + 128) // 2
    assert fpq.fpq_conv2d_split_workspace_size(2, 320, 300, 8, 8, 16, 3, 3, 1, 1, fpq.E4M3, fpq.E4M3) == 2 * 100 * (384 + 304)
    assert fpq.fpq_conv2d_split_workspace_size(2, 0, 300, 8, 8, 16, 3, 3, 1, 1, fpq.E4M3, fpq.E4M3) == 0
