"""Parity of the quantized linear / conv layers (CUDA, through the C ABI) with the CPU oracle.

Acceptance per output element: |err| <= 1e-3 * sum_k |a_k b_k| (+ 2 FP32 ulps of |y|
for the final scale-and-bias rounding); the weight codes must match bit for bit.
"""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2408_06995_b200 as fpq
from paper_2408_06995_b200 import inputs as I
from _helpers import FMT, Guarded, assert_close, gpu_layer, gpu_prepare, layer_scales, oracle_layer, sample_indices

pytestmark = pytest.mark.gpu


def _check_full(L, use_bias=True):
    ws, xs = layer_scales(L)
    y = gpu_layer(L, ws, xs, use_bias)
    yr, ab = oracle_layer(L, ws, xs, None, use_bias)
    assert y.shape == yr.shape
    return assert_close(y, yr, ab)


def _tile_edges(L):
    """Flat output indices of the first and last 128 rows (all columns) and of the first and last 128
    columns (all rows) of the layer seen as an M x N matrix: the edge tiles of the contraction."""
    M, N = L.M, L.N
    rows = np.unique(np.concatenate([np.arange(min(128, M)), np.arange(max(0, M - 128), M)]))
    cols = np.unique(np.concatenate([np.arange(min(128, N)), np.arange(max(0, N - 128), N)]))
    if L.kind == "linear":
        a = (rows[:, None] * N + np.arange(N)[None, :]).reshape(-1)
        b = (np.arange(M)[:, None] * N + cols[None, :]).reshape(-1)
    else:
        hw = L.Ho * L.Wo                                   # row m = (image, pixel); NCHW output
        def flat(m, n):
            return (m // hw) * (N * hw) + n * hw + (m % hw)
        a = flat(rows[:, None], np.arange(N)[None, :]).reshape(-1)
        b = flat(np.arange(M)[:, None], cols[None, :]).reshape(-1)
    return np.concatenate([a, b]).astype(np.int64)


def _check_sampled(L, nsamp, seed, full_limit=1 << 22):
    """Every output element where the layer has at most full_limit of them; otherwise nsamp seeded random
    elements plus every element of the first and last tile row and tile column."""
    ws, xs = layer_scales(L)
    y = gpu_layer(L, ws, xs)
    assert np.all(np.isfinite(y))
    total = y.size
    if total <= full_limit:
        yr, ab = oracle_layer(L, ws, xs)
        return assert_close(y, yr, ab)
    idx = sample_indices(total, nsamp, seed, _tile_edges(L))
    yr, ab = oracle_layer(L, ws, xs, idx)
    return assert_close(y.reshape(-1)[idx], yr, ab)


# ---- linear ------------------------------------------------------------------------------

def test_config1_linear_w8a8_every_element():
    (L,) = I.config1()
    _check_full(L)


@pytest.mark.parametrize("wfmt", ["e4m3", "e2m1"])
@pytest.mark.parametrize("M,K,N", [(1, 16, 1), (2, 1280, 320), (127, 128, 64), (128, 128, 128), (129, 129, 129),
                                   (130, 200, 72), (154, 768, 640), (300, 320, 960), (257, 1000, 4), (64, 48, 260)])
def test_linear_ragged_shapes(wfmt, M, K, N):
    L = I.linear_layer("t", M, K, N, wfmt, rounding=(wfmt == "e2m1"))
    I.draw(L, 7, M + K + N, "normal", 0.02, True, 0.01, (0.001, 20.0))
    _check_full(L)
    _check_full(L, use_bias=False)


def test_same_addresses_other_shapes():
    """Layers of different shapes called one after the other on the same device addresses (one arena for inputs,
    scratch and outputs, as a network's allocator would hand out): the library remembers the TMA descriptors it
    has made per (address, shape), so a descriptor of an earlier shape at the same address must never be taken.
    Every result must equal, bit for bit, the one computed in buffers of its own."""
    shapes = [(300, 320, 960), (300, 960, 320), (150, 640, 960), (300, 320, 960), (256, 128, 128), (128, 128, 256)]
    arena_x = torch.empty(1 << 20, dtype=torch.float32, device="cuda")
    arena_y = torch.empty(1 << 20, dtype=torch.float32, device="cuda")
    arena_w = torch.empty(4 << 20, dtype=torch.uint8, device="cuda")
    arena_p = torch.empty(1 << 20, dtype=torch.uint8, device="cuda")
    for wfmt in ("e4m3", "e2m1"):
        gfw, _ = FMT[wfmt]
        for j, (M, K, N) in enumerate(shapes):
            L = I.linear_layer("t", M, K, N, wfmt, rounding=False)
            I.draw(L, 9, 10 * j, "normal", 0.02, True, 0.01)
            ws, xs = layer_scales(L)
            want = gpu_layer(L, ws, xs)
            codes = fpq.fpq_quantize_weight(torch.from_numpy(L.w.reshape(N, K)).cuda(), torch.from_numpy(ws).cuda(), gfw, None)
            nprep = fpq.fpq_prepared_size(gfw, fpq.LINEAR, N, K)
            prep = fpq.fpq_prepare_weight(codes, gfw, fpq.LINEAR, N, K, prepared=arena_p[:nprep])
            x = arena_x[:M * K].view(M, K)
            x.copy_(torch.from_numpy(L.x))
            y = arena_y[:M * N].view(M, N)
            nws = max(256, fpq.fpq_linear_workspace_size(M, N, K, fpq.E4M3, gfw))
            fpq.fpq_linear(x, prep, torch.from_numpy(ws).cuda(), xs, fpq.E4M3, gfw, torch.from_numpy(L.bias).cuda(), N, y=y,
                           workspace=arena_w[:nws])
            assert fpq.fpq_read_status() == fpq.OK
            assert np.array_equal(y.cpu().numpy(), want), (wfmt, M, K, N)


# at most 8 rows: one pass over the weights on the CUDA cores instead of the tensor-core kernel
@pytest.mark.parametrize("wfmt", ["e4m3", "e2m1"])
@pytest.mark.parametrize("M,K,N", [(1, 128, 8), (2, 320, 1280), (3, 1000, 77), (8, 1280, 320), (8, 3072, 40), (5, 130, 1),
                                   (8, 3200, 16), (4, 5120, 130)])   # K = 130 is not a multiple of 4: tensor-core path
def test_linear_few_rows(wfmt, M, K, N):
    L = I.linear_layer("t", M, K, N, wfmt, rounding=(wfmt == "e2m1"))
    I.draw(L, 15, M + K + N, "normal", 0.02, True, 0.01, (0.01, 20.0))
    _check_full(L)


@pytest.mark.parametrize("wfmt", ["e4m3", "e2m1"])
def test_linear_small_integers_are_exact(wfmt):
    rng = np.random.default_rng(3)
    M, K, N = 200, 384, 136
    ints = np.array([0, 1, 2, -1, -2, 4, -4], dtype=np.float32)
    L = I.linear_layer("ints", M, K, N, wfmt)
    L.x = ints[rng.integers(0, 7, (M, K))]
    L.w = ints[rng.integers(0, 7, (N, K))]
    L.bias = np.zeros(N, np.float32)
    ws = np.ones(N, np.float32)
    y = gpu_layer(L, ws, 1.0)
    assert np.array_equal(y.astype(np.float64), L.x.astype(np.float64) @ L.w.astype(np.float64).T)


def test_weight_codes_and_prepared_copy_are_bit_exact():
    for wfmt, C, R in (("e4m3", 20, 3), ("e2m1", 20, 3), ("e2m1", 130, 1), ("e4m3", 7, 3), ("e2m1", 7, 3)):
        L = I.conv_layer("w", 1, C, 8, 8, 10, R, wfmt=wfmt, rounding=True)
        I.draw(L, 8, C + R, "normal", 0.05, True)
        ws, xs = layer_scales(L)
        gfw, ofw = FMT[wfmt]
        codes, prep = gpu_prepare(L, ws)
        want = O.quantize_weight(L.w.reshape(L.N, -1), ws, ofw, O.pack_bits(L.bits))
        assert np.array_equal(codes.cpu().numpy(), want)
        # prepared copy: [N][R*S][C_pad], taps outermost, zero padded
        K = C * R * R
        flat = want if ofw.bits == 8 else np.stack([want & 15, want >> 4], -1).reshape(L.N, -1)[:, :K]
        Cp = (C + 127) // 128 * 128
        exp = np.zeros((L.N, R * R, Cp), np.uint8)
        exp[:, :, :C] = flat.reshape(L.N, C, R * R).transpose(0, 2, 1)
        if ofw.bits == 4:
            e2 = exp.reshape(L.N, -1)
            exp = (e2[:, 0::2] | (e2[:, 1::2] << 4)).astype(np.uint8)
        assert np.array_equal(prep.cpu().numpy().reshape(L.N, -1), exp.reshape(L.N, -1))


# ---- conv ---------------------------------------------------------------------------------

@pytest.mark.parametrize("wfmt", ["e4m3", "e2m1"])
@pytest.mark.parametrize("B,C,H,W,Co,R,pad,stride", [
    (1, 16, 8, 8, 16, 3, 1, 1),
    (2, 4, 16, 16, 8, 3, 1, 1),        # fewer channels than one 16-byte row
    (3, 20, 9, 7, 5, 3, 1, 1),         # odd extents, ragged everything
    (2, 32, 16, 16, 24, 3, 1, 2),      # stride 2
    (1, 8, 11, 13, 6, 3, 1, 2),
    (2, 130, 8, 8, 140, 1, 0, 1),      # 1x1, channels just past a chunk
    (1, 64, 32, 32, 64, 3, 1, 1),
    (2, 16, 64, 64, 4, 3, 1, 1),       # conv_out-like
    (1, 8, 5, 5, 8, 3, 0, 1),          # no padding
    (5, 12, 4, 4, 260, 3, 1, 1),       # several images per tile, three N tiles
])
def test_conv_ragged_shapes(wfmt, B, C, H, W, Co, R, pad, stride):
    L = I.conv_layer("t", B, C, H, W, Co, R, pad=pad, stride=stride, wfmt=wfmt, rounding=True)
    I.draw(L, 9, B + C + H + Co, "silu", 0.03, True)
    _check_full(L)


# few output tiles and a long reduction: the kernel splits the reduction over a cluster of CTAs
@pytest.mark.parametrize("wfmt", ["e4m3", "e2m1"])
@pytest.mark.parametrize("B,C,H,W,Co,R,pad,stride", [
    (2, 640, 8, 8, 200, 3, 1, 1),      # 5 chunks, 2 x 2 tiles
    (1, 1100, 8, 8, 130, 3, 1, 1),     # 9 chunks, the last one ragged; unequal ranges
    (2, 300, 16, 16, 96, 3, 1, 2),     # stride 2, 3 chunks
    (2, 520, 8, 8, 260, 1, 0, 1),      # 1x1, 5 chunks, three column tiles
    (1, 256, 4, 4, 8, 3, 1, 1),        # 64-column tiles
])
def test_conv_split_reduction_shapes(wfmt, B, C, H, W, Co, R, pad, stride):
    L = I.conv_layer("t", B, C, H, W, Co, R, pad=pad, stride=stride, wfmt=wfmt, rounding=True)
    I.draw(L, 12, B + C + H + Co, "silu", 0.03, True)
    _check_full(L)


def test_conv_paired_row_tiles_every_element():
    # more 3x3 tiles than SMs with streamed weights: the kernel walks pairs of row tiles that share
    # each weight stage (154 tiles, the last pair is half empty)
    L = I.conv_layer("t", 17, 256, 32, 32, 128, 3, wfmt="e2m1", rounding=True)
    I.draw(L, 14, 0, "silu", 0.03, True)
    _check_full(L)


def test_conv_1x1_matches_linear_on_the_gpu():
    L = I.conv_layer("c", 2, 96, 8, 8, 80, 1, wfmt="e4m3")
    I.draw(L, 10, 0, "normal", 0.02, True)
    ws, xs = layer_scales(L)
    yc = gpu_layer(L, ws, xs)
    Ll = I.linear_layer("l", 2 * 64, 96, 80, "e4m3")
    Ll.x = np.ascontiguousarray(L.x.transpose(0, 2, 3, 1).reshape(-1, 96))
    Ll.w = L.w.reshape(80, 96)
    Ll.bias = L.bias
    yl = gpu_layer(Ll, ws, xs)
    assert np.array_equal(yc.transpose(0, 2, 3, 1).reshape(-1, 80), yl)


def test_conv_one_hot_tap_is_a_shift():
    B, C, H, W = 2, 16, 8, 8
    L = I.conv_layer("s", B, C, H, W, 1, 3, wfmt="e4m3")
    I.draw(L, 11, 0, "normal", 0.02)
    L.bias[:] = 0
    xs = O.scale_from_max(np.abs(L.x).max(), O.E4M3)
    xq = O.decode_table(O.E4M3)[O.quantize_act(L.x, xs, O.E4M3)] * np.float64(xs)
    for r, s in [(0, 0), (1, 2), (2, 1), (1, 1)]:
        L.w[:] = 0
        L.w[0, 5, r, s] = 1.0
        y = gpu_layer(L, np.ones(1, np.float32), float(xs))
        want = np.zeros((B, H, W))
        ys, xsl = slice(max(0, 1 - r), min(H, H + 1 - r)), slice(max(0, 1 - s), min(W, W + 1 - s))
        for oy in range(H):
            for ox in range(W):
                iy, ix = oy + r - 1, ox + s - 1
                if 0 <= iy < H and 0 <= ix < W:
                    want[:, oy, ox] = xq[:, 5, iy, ix]
        assert np.allclose(y[:, 0], want, rtol=3e-7, atol=0)


def test_config2_conv_w8a8_reduced_batch_every_element():
    (L,) = I.config2(batch=4)
    _check_full(L)


def test_config3_pair_w4a8_reduced_batch_every_element():
    for L in I.config3(batch=2):
        _check_full(L)


# ---- full sizes, sampled outputs ---------------------------------------------------------

def test_config2_full_size_every_element():
    # the workload the bench times, in its launch configuration (several tiles per CTA, double-buffered walk)
    (L,) = I.config2()
    _check_sampled(L, 0, 1, full_limit=1 << 24)


def test_config3_full_size():
    # conv 3x3 256 -> 256: every element; conv 1x1 256 -> 512: 2^20 samples and the edge tiles
    for j, L in enumerate(I.config3()):
        _check_sampled(L, 1 << 20, 2 + j)


def test_config4_full_size():
    # out-projection and FFN-out: every element; QKV and GEGLU: 2^20 samples and the edge tiles
    for j, L in enumerate(I.config4()):
        _check_sampled(L, 1 << 20, 10 + j)


def _sd_shapes():
    out = []
    for item in I.distinct_shapes(I.sd_v1_unet_layers()):
        out.append(item[0] if isinstance(item, tuple) else item)
    return out


@pytest.mark.parametrize("j", range(58))
def test_config5_every_sd_unet_shape_sampled(j):
    # all distinct conv / linear shapes of one SD-v1-style U-Net step (W4A8 with rounding decisions),
    # at the sizes and in the launch configuration the bench times; the oracle checks a sample
    shapes = _sd_shapes()
    assert len(shapes) == 58
    L = shapes[j]
    I.draw(L, 5, 10 * j, "normal", 0.02, True)
    # every element up to 2^22 outputs, else 2^16 samples and the edge tiles
    _check_sampled(L, 1 << 16, 100 + j)


# ---- the two-kernel route (activation codes in a workspace, then the contraction) ---------------

def _staged(L, ws, xs):
    gfw, _ = FMT[L.wfmt]
    _, prep = gpu_prepare(L, ws)
    x = torch.from_numpy(L.x).cuda()
    bias = torch.from_numpy(L.bias).cuda()
    wsd = torch.from_numpy(ws).cuda()
    if L.kind == "linear":
        wk = torch.empty(max(1, fpq.fpq_linear_workspace_size(L.M, L.N, L.K, fpq.E4M3, gfw)), dtype=torch.uint8, device="cuda")
        y = torch.empty((L.M, L.N), dtype=torch.float32, device="cuda")
        fpq.fpq_linear_quantize_input(x, xs, fpq.E4M3, gfw, L.N, wk)
        fpq.fpq_linear_contract(wk, prep, wsd, xs, fpq.E4M3, gfw, bias, y, L.K)
    else:
        wk = torch.empty(max(1, fpq.fpq_conv2d_workspace_size(L.B, L.C, L.H, L.W, L.N, L.R, L.S, L.pad, L.stride,
                                                               fpq.E4M3, gfw)), dtype=torch.uint8, device="cuda")
        y = torch.empty((L.B, L.N, L.Ho, L.Wo), dtype=torch.float32, device="cuda")
        fpq.fpq_conv2d_quantize_input(x, xs, fpq.E4M3, gfw, L.N, L.R, L.S, L.pad, L.stride, wk)
        fpq.fpq_conv2d_contract(wk, prep, wsd, xs, fpq.E4M3, gfw, bias, y, (L.B, L.C, L.H, L.W), L.R, L.S, L.pad, L.stride)
    assert fpq.fpq_read_status() == fpq.OK
    return y.cpu().numpy(), wk.cpu().numpy()


@pytest.mark.parametrize("wfmt", ["e4m3", "e2m1"])
def test_two_kernel_route_matches_the_oracle_and_the_fused_call(wfmt):
    layers = [
        I.draw(I.linear_layer("l", 300, 320, 200, wfmt, rounding=True), 13, 0, "normal", 0.02, True),
        I.draw(I.linear_layer("l2", 130, 1000, 72, wfmt), 13, 10, "normal", 0.02, True),
        I.draw(I.conv_layer("c", 3, 20, 9, 7, 37, 3, wfmt=wfmt, rounding=True), 13, 20, "silu", 0.03, True),
        I.draw(I.conv_layer("c2", 2, 130, 16, 16, 140, 1, wfmt=wfmt), 13, 30, "silu", 0.03, True),
        I.draw(I.conv_layer("c3", 2, 32, 16, 16, 24, 3, stride=2, wfmt=wfmt), 13, 40, "silu", 0.03, True),
    ]
    for L in layers:
        ws, xs = layer_scales(L)
        y2, codes = _staged(L, ws, xs)
        yr, ab = oracle_layer(L, ws, xs)
        assert_close(y2, yr, ab)
        assert np.array_equal(y2, gpu_layer(L, ws, xs, route="two"))      # same kernels, same order
        # the codes in the workspace are the oracle's, in the operand layout
        want = O.quantize_act(L.x, xs, O.E4M3)
        if L.kind == "linear":
            Kp = (L.K + 15) // 16 * 16
            got = codes[: L.M * Kp].reshape(L.M, Kp)
            assert np.array_equal(got[:, : L.K], want) and not got[:, L.K:].any()
        else:
            Cp = (L.C + 15) // 16 * 16
            Hp, Wp = L.H + 2 * L.pad, L.W + 2 * L.pad
            got = codes[: L.B * Hp * Wp * Cp].reshape(L.B, Hp, Wp, Cp)
            inner = got[:, L.pad:L.pad + L.H, L.pad:L.pad + L.W, : L.C]
            assert np.array_equal(inner, want.transpose(0, 2, 3, 1))
            assert got.sum() == inner.sum()                    # frame and channel padding are code 0


# ---- host-buffer forms (copy in, layer, copy out; pipelined in slices when the batch is large) ----------

@pytest.mark.parametrize("kind,shape", [
    ("conv", (16, 64, 32, 32, 64, 3)),        # 8 MiB of copies: eight slices of two images
    ("conv", (3, 20, 9, 7, 37, 3)),           # small: one slice
    ("conv", (5, 130, 32, 32, 140, 1)),       # 5 images in 5 slices
    ("linear", (4096, 320, 320)),             # sliced by rows
    ("linear", (3000, 640, 200)),             # 3000 rows in 8 unequal slices
    ("linear", (4096, 130, 322)),             # rows are not 16-byte multiples: one slice
])
def test_host_forms_equal_the_device_forms(kind, shape):
    if kind == "conv":
        B, C, H, W, Co, R = shape
        L = I.conv_layer("h", B, C, H, W, Co, R, wfmt="e4m3", rounding=True)
    else:
        M, K, N = shape
        L = I.linear_layer("h", M, K, N, "e2m1", rounding=True)
    I.draw(L, 16, sum(shape), "normal", 0.02, True)
    ws, xs = layer_scales(L)
    gfw, _ = FMT[L.wfmt]
    _, prep = gpu_prepare(L, ws)
    want = gpu_layer(L, ws, xs)
    xh = torch.from_numpy(L.x).pin_memory()
    xd = torch.empty_like(xh, device="cuda")
    wsd = torch.from_numpy(ws).cuda()
    bias = torch.from_numpy(L.bias).cuda()
    if kind == "conv":
        yg = Guarded(4 * L.B * L.N * L.Ho * L.Wo)
        yd = yg.f32((L.B, L.N, L.Ho, L.Wo))
        wg = Guarded(fpq.fpq_conv2d_workspace_size(L.B, L.C, L.H, L.W, L.N, L.R, L.S, L.pad, L.stride, fpq.E4M3, gfw))
    else:
        yg = Guarded(4 * L.M * L.N)
        yd = yg.f32((L.M, L.N))
        wg = Guarded(max(1, fpq.fpq_linear_workspace_size(L.M, L.N, L.K, fpq.E4M3, gfw)))
    wk = wg.inner
    yh = torch.empty(yd.shape, dtype=torch.float32).pin_memory()
    for _ in range(2):                                    # twice: the pipeline's streams and events are reused
        yh.fill_(float("nan"))
        if kind == "conv":
            fpq.fpq_conv2d_host(xh, xd, prep, wsd, xs, fpq.E4M3, gfw, bias, yd, yh, L.R, L.S, L.pad, L.stride, wk)
        else:
            fpq.fpq_linear_host(xh, xd, prep, wsd, xs, fpq.E4M3, gfw, bias, yd, yh, wk)
        assert fpq.fpq_read_status() == fpq.OK
        assert np.array_equal(yh.numpy(), want)
        yg.check("host form: device output")
        wg.check("host form: workspace")
