"""Bit-exact parity of the CUDA quantizer with the CPU oracle (through the C ABI)."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2408_06995_b200 as fpq
from _helpers import to_oracle

pytestmark = pytest.mark.gpu

FORMATS = [fpq.E4M3, fpq.Format(4, 3, 7, fpq.SAT_PAPER), fpq.Format(4, 3, 8), fpq.E5M2, fpq.Format(5, 2, 16),
           fpq.E3M4, fpq.E2M5, fpq.E2M1, fpq.Format(2, 1, 2), fpq.E1M2]


def _unpack(codes, K):
    c = np.stack([codes & 15, codes >> 4], axis=-1).reshape(codes.shape[0], -1)
    return c[:, :K]


def _sweep(f):
    of = to_oracle(f)
    tab = O.decode_table(of)
    g = np.unique(np.abs(tab))
    pts = list(g) + list((g[1:] + g[:-1]) / 2) + [g.max() * 1.01, g.max() * 7, 1e30, np.inf, 1e-30, 1e-42, 0.0]
    pts = np.array(pts, dtype=np.float32)
    pts = np.concatenate([pts, np.nextafter(pts, np.float32(np.inf)), np.nextafter(pts, np.float32(-np.inf))])
    pts = np.concatenate([pts, -pts])
    return pts[~np.isnan(pts)]


@pytest.mark.parametrize("f", FORMATS)
def test_weight_encode_sweep_all_modes(f):
    of = to_oracle(f)
    pts = _sweep(f)
    for scale, pad16 in ((1.0, False), (0.25, True), (0.0371, True), (3.3, False)):
        x = (pts * np.float32(scale)).astype(np.float32)
        if pad16:       # rows of a multiple of 16 weights take the 16-per-thread kernels
            x = np.concatenate([x, np.zeros(-x.size % 16, np.float32)])
        N = 3
        K = x.size
        w = np.stack([x, x[::-1], np.roll(x, 5)]).astype(np.float32)
        sc = np.array([scale, scale * 2, scale * 0.77], dtype=np.float32)
        rng = np.random.default_rng(5)
        for bits in (None, np.zeros((N, K), np.uint8), np.ones((N, K), np.uint8),
                     rng.integers(0, 2, (N, K), dtype=np.uint8)):
            rb = None if bits is None else O.pack_bits(bits)
            want = O.quantize_weight(w, sc, of, rb)
            got = fpq.fpq_quantize_weight(torch.from_numpy(w).cuda(), torch.from_numpy(sc).cuda(), f,
                                          None if rb is None else torch.from_numpy(rb).cuda()).cpu().numpy()
            assert np.array_equal(got, want), (f, scale, bits is None)
    fpq.fpq_read_status()   # the sweep contains no NaN, but clear anyway


@pytest.mark.parametrize("f", FORMATS)
@pytest.mark.parametrize("shape", [(1, 1), (5, 7), (3, 16), (2, 33), (64, 1152), (7, 1001)])
def test_weight_encode_random(f, shape):
    of = to_oracle(f)
    N, K = shape
    rng = np.random.default_rng(N * 1000 + K)
    w = (rng.standard_normal((N, K)) * 0.02 * rng.uniform(0.5, 2, (N, 1))).astype(np.float32)
    sc = np.array([O.scale_from_max(np.abs(r).max(), of) for r in w], dtype=np.float32)
    bits = rng.integers(0, 2, (N, K), dtype=np.uint8)
    for rb in (None, O.pack_bits(bits)):
        want = O.quantize_weight(w, sc, of, rb)
        got = fpq.fpq_quantize_weight(torch.from_numpy(w).cuda(), torch.from_numpy(sc).cuda(), f,
                                      None if rb is None else torch.from_numpy(rb).cuda()).cpu().numpy()
        assert got.shape == want.shape
        assert np.array_equal(got, want)


@pytest.mark.parametrize("f", FORMATS)
@pytest.mark.parametrize("n", [1, 15, 16, 17, 4096 + 7, 300001])
def test_act_quantize_random(f, n):
    of = to_oracle(f)
    rng = np.random.default_rng(n)
    x = rng.standard_normal(n).astype(np.float32)
    x[rng.integers(0, n, max(1, n // 1000))] *= 20
    scale = O.scale_from_max(np.abs(x).max() * 0.8, of)     # some values clip
    want = O.quantize_act(x, scale, of)
    got = fpq.fpq_quantize_act(torch.from_numpy(x).cuda(), float(scale), f).cpu().numpy()
    assert np.array_equal(got.reshape(-1), want.reshape(-1))
    # a view that starts 4 bytes into an allocation takes the unaligned path
    xd = torch.zeros(n + 1, dtype=torch.float32, device="cuda")
    xd[1:] = torch.from_numpy(x).cuda()
    got2 = fpq.fpq_quantize_act(xd[1:], float(scale), f).cpu().numpy()
    assert np.array_equal(got2.reshape(-1), want.reshape(-1))


@pytest.mark.parametrize("f", FORMATS)
def test_act_quantize_sweep(f):
    """Every grid value, every tie and their FP32 neighbours, both signs (the hardware-convert kernels of E4M3, the
    OCP E5M2 and E2M1 and the general arithmetic alike)."""
    pts = _sweep(f)
    for scale in (1.0, 0.5, 0.0371, 11.0):
        x = np.tile((pts * np.float32(scale)).astype(np.float32), 3)
        want = O.quantize_act(x, scale, to_oracle(f))
        got = fpq.fpq_quantize_act(torch.from_numpy(x).cuda(), scale, f).cpu().numpy()
        assert np.array_equal(got.reshape(-1), want.reshape(-1))


@pytest.mark.parametrize("f", [fpq.Format(4, 3, -91), fpq.Format(4, 3, 123), fpq.Format(2, 1, -101), fpq.Format(2, 1, 125),
                               fpq.Format(1, 6, -108), fpq.Format(1, 6, 120)])
def test_exponent_bias_at_the_ends_of_its_range(f):
    """The smallest and largest exponent bias the library accepts: grid values next to the ends of FP32's normal
    range, flat quantizer and weight encoder (nearest and learned), 16-per-thread kernels."""
    of = to_oracle(f)
    pts = _sweep(f)
    pts = pts[np.isfinite(pts)]
    x = np.concatenate([pts, np.zeros(-pts.size % 16, np.float32)])
    want = O.quantize_act(x, 1.0, of)
    got = fpq.fpq_quantize_act(torch.from_numpy(x).cuda(), 1.0, f).cpu().numpy()
    assert np.array_equal(got.reshape(-1), want.reshape(-1))
    w = np.stack([x, x[::-1]]).astype(np.float32)
    sc = np.ones(2, np.float32)
    rng = np.random.default_rng(11)
    for rb in (None, O.pack_bits(rng.integers(0, 2, w.shape, dtype=np.uint8))):
        got = fpq.fpq_quantize_weight(torch.from_numpy(w).cuda(), torch.from_numpy(sc).cuda(), f,
                                      None if rb is None else torch.from_numpy(rb).cuda()).cpu().numpy()
        assert np.array_equal(got, O.quantize_weight(w, sc, of, rb))
    assert fpq.fpq_read_status() == fpq.OK


def test_special_values_and_status_flag():
    assert fpq.fpq_read_status() == fpq.OK
    x = np.zeros(64, dtype=np.float32)
    x[3], x[4], x[5], x[6], x[20] = np.inf, -np.inf, -0.0, -1e-30, 1.0
    for f in (fpq.E4M3, fpq.E5M2, fpq.E2M1, fpq.E3M4):
        got = fpq.fpq_quantize_act(torch.from_numpy(x).cuda(), 1.0, f).cpu().numpy()
        want = O.quantize_act(x, 1.0, to_oracle(f))
        assert np.array_equal(got.reshape(-1), want.reshape(-1))
        assert fpq.fpq_read_status() == fpq.OK
    x[7] = x[40] = x[41] = np.nan
    for f in (fpq.E4M3, fpq.E5M2, fpq.E2M1, fpq.E3M4):
        got = fpq.fpq_quantize_act(torch.from_numpy(x).cuda(), 1.0, f).cpu().numpy()
        want = O.quantize_act(x, 1.0, to_oracle(f))
        assert np.array_equal(got.reshape(-1), want.reshape(-1))
        if f is not fpq.E2M1:
            assert got[7] == 0
        assert fpq.fpq_read_status() == fpq.ERR_NAN_INPUT
        assert fpq.fpq_read_status() == fpq.OK          # reading clears it
    # the weight encoders: rows of 64 (16 per thread) and of 63 (8 per thread), with and without rounding decisions
    for f in (fpq.E4M3, fpq.E5M2, fpq.E2M1, fpq.E3M4):
        for K in (64, 63):
            w = np.stack([x[:K], x[:K][::-1]]).astype(np.float32)
            sc = np.ones(2, np.float32)
            for rb in (None, O.pack_bits(np.ones((2, K), np.uint8))):
                got = fpq.fpq_quantize_weight(torch.from_numpy(w).cuda(), torch.from_numpy(sc).cuda(), f,
                                              None if rb is None else torch.from_numpy(rb).cuda()).cpu().numpy()
                assert np.array_equal(got, O.quantize_weight(w, sc, to_oracle(f), rb))
                assert fpq.fpq_read_status() == fpq.ERR_NAN_INPUT


def test_empty_inputs():
    x = torch.empty(0, dtype=torch.float32, device="cuda")
    assert fpq.fpq_quantize_act(x, 1.0, fpq.E4M3).numel() == 0
    w = torch.empty((0, 8), dtype=torch.float32, device="cuda")
    assert fpq.fpq_quantize_weight(w, torch.empty(0, device="cuda"), fpq.E4M3).numel() == 0


def test_full_size_activation_tensor_sampled():
    """The standalone quantizer on a tensor the size of the DDIM-style conv input
    (64 x 128 x 32 x 32): every code compared."""
    rng = np.random.default_rng(2000)
    x = rng.standard_normal(64 * 128 * 32 * 32, dtype=np.float32)
    x = (x / (1 + np.exp(-x))).astype(np.float32)
    scale = O.scale_from_max(np.abs(x).max(), O.E4M3)
    got = fpq.fpq_quantize_act(torch.from_numpy(x).cuda(), float(scale), fpq.E4M3).cpu().numpy()
    want = O.quantize_act(x, scale, O.E4M3)
    assert np.array_equal(got, want)


@pytest.mark.parametrize("fname", ["E4M3", "E2M1", "E3M4", "E1M2"])
@pytest.mark.parametrize("n", [0, 1, 15, 16, 33, 4097, 1 << 20, (1 << 20) + 3])
def test_zero_census_matches_the_oracle(fname, n):
    fo, fg = getattr(O, fname), getattr(fpq, fname)
    rng = np.random.default_rng(n + 17)
    x = (rng.standard_normal(n) * 0.3).astype(np.float32)
    x[rng.random(n) < 0.1] = 0.0
    scale = 0.4 if fo.bits == 8 else 0.2
    codes = O.quantize_act(x, scale, fo).reshape(-1)
    # one byte of offset: the kernel must cope with a start that is not 16-byte aligned
    buf = torch.zeros(codes.size + 1, dtype=torch.uint8, device="cuda")
    buf[1:] = torch.from_numpy(codes).cuda()
    for view in (buf[1:], buf[1:].clone()):
        got = int(fpq.fpq_zero_census(view, n, fg).cpu()[0])
        assert got == O.zero_count(codes, n, fo)
