"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests compares the oracle with itself: the expected values are
closed forms worked by hand (tests/golden), brute-force searches over an
independently built grid, PyTorch's own FP8 casts, numpy/torch float64
contractions, or structural invariants.
"""
import os

import numpy as np
import pytest
import torch

import oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")
PAPER_FORMATS = [O.E2M5, O.E3M4, O.Format(4, 3, 8), O.Format(4, 3, 7), O.E4M3, O.Format(5, 2, 16),
                 O.E5M2, O.E1M2, O.Format(2, 1, 2), O.E2M1]


def _rows(name):
    with open(os.path.join(GOLD, name)) as fh:
        for line in fh:
            line = line.strip()
            if line and not line.startswith("#"):
                yield line.split()


# ---- format ------------------------------------------------------------------

def test_format_constants_closed_form():
    for e, m, b, sat, cm, msub, mnorm in _rows("format_constants.txt"):
        f = O.Format(int(e), int(m), int(b), int(sat))
        assert O.cmax(f) == float(cm)
        tab = O.decode_table(f)
        pos = np.unique(tab[tab > 0])
        assert pos[0] == float(msub)
        assert O.decode(1 << f.m, f) == float(mnorm)
        # with every exponent finite the largest code is the clipping value
        assert tab.max() == O.cmax(O.Format(f.e, f.m, f.B, O.SAT_PAPER))


def test_explicit_small_grids():
    tab = O.decode_table(O.E2M1)
    assert list(tab[:8]) == [0, 0.5, 1, 1.5, 2, 3, 4, 6]
    assert list(tab[8:]) == [-0.0, -0.5, -1, -1.5, -2, -3, -4, -6]
    # E1M2 with bias 1 is a uniform grid of step 1/4 (the paper's integer quantizer in sign-magnitude form)
    tab = O.decode_table(O.E1M2)
    assert list(tab[:8]) == [0.25 * i for i in range(8)]


def test_decode_matches_torch_fp8_tables():
    codes = torch.arange(256, dtype=torch.uint8)
    t43 = codes.view(torch.float8_e4m3fn).float().numpy().astype(np.float64)
    t52 = codes.view(torch.float8_e5m2).float().numpy().astype(np.float64)
    o43 = O.decode_table(O.E4M3)
    o52 = O.decode_table(O.E5M2)
    ok43 = np.isfinite(t43)
    assert ok43.sum() == 254
    assert np.array_equal(o43[ok43], t43[ok43])
    ok52 = np.isfinite(t52)
    assert ok52.sum() == 248
    assert np.array_equal(o52[ok52], t52[ok52])
    # the codes the OCP types reserve are finite in the paper's format
    assert o43[0x7F] == 480.0 and o52[0x7C] == 65536.0


def test_grid_is_strictly_increasing_in_code():
    for f in PAPER_FORMATS:
        half = O.decode_table(f)[: 1 << (f.e + f.m)]
        assert np.all(np.diff(half) > 0)


@pytest.mark.parametrize("f", PAPER_FORMATS)
def test_every_code_is_a_fixed_point(f):
    tab = O.decode_table(f)
    cm = O.cmax(f)
    for code, v in enumerate(tab):
        if abs(v) > cm:
            continue  # not produced in NATIVE saturation
        want = 0 if v == 0 else code
        assert O.quantize_one(v, 1.0, f, -1) == want
        assert O.quantize_one(v, 1.0, f, 0) == want


# ---- brute force --------------------------------------------------------------

def _grid(f):
    """Signed grid built from the format equation, independent of the oracle:
    returns sorted values and the magnitude-code of each."""
    vals = []
    for p in range(1 << f.e):
        for d in range(1 << f.m):
            if p == 0:
                v = d * 2.0 ** (1 - f.B - f.m)
            else:
                v = 2.0 ** (p - f.B) * (1 + d / 2.0 ** f.m)
            vals.append(v)
    vals = np.array(vals)
    cm = (2 - 2.0 ** -f.m) * 2.0 ** (2 ** f.e - f.B - 1)
    if f.sat == O.SAT_NATIVE and (f.e, f.m) == (4, 3):
        cm = 1.75 * 2.0 ** (15 - f.B)
    if f.sat == O.SAT_NATIVE and (f.e, f.m) == (5, 2):
        cm = 1.75 * 2.0 ** (30 - f.B)
    return vals[vals <= cm], cm


def _sweep_points(f):
    g, cm = _grid(f)
    pts = list(g) + list((g[1:] + g[:-1]) / 2)
    pts += [cm * 1.01, cm * 4, 1e30, np.inf, 1e-30, 1e-42, 0.0]
    pts = np.array(pts, dtype=np.float32)
    pts = np.concatenate([pts, np.nextafter(pts, np.float32(np.inf)), np.nextafter(pts, np.float32(-np.inf))])
    pts = np.concatenate([pts, -pts])
    return pts[~np.isnan(pts)]


def _brute_rtn(t, f):
    g, cm = _grid(f)
    a = min(max(float(t), -cm), cm)
    d = np.abs(g - abs(a))
    best = d.min()
    cand = np.nonzero(d == best)[0]
    if len(cand) == 2:  # tie: even code (even mantissa LSB; a power of two has mantissa 0)
        idx = cand[0] if cand[0] % 2 == 0 else cand[1]
    else:
        idx = cand[0]
    if g[idx] == 0:
        return 0
    return int(idx) | ((1 << (f.e + f.m)) if a < 0 else 0)


@pytest.mark.parametrize("f", PAPER_FORMATS)
def test_rtn_equals_nearest_grid_point_ties_to_even(f):
    for t in _sweep_points(f):
        assert O.quantize_one(t, 1.0, f, -1) == _brute_rtn(t, f), (f, t)


@pytest.mark.parametrize("f", [O.E4M3, O.E2M1, O.E3M4])
def test_rtn_with_power_of_two_scales(f):
    # x / 2^j is exact, so the result is the brute-force answer on x / 2^j
    for j in (-3, 5):
        sc = 2.0 ** j
        for t in _sweep_points(f)[::3]:
            x = np.float32(t) * np.float32(sc)
            if not np.isfinite(x) and np.isfinite(t):
                continue
            assert O.quantize_one(x, sc, f, -1) == _brute_rtn(np.float32(x) / np.float32(sc), f)


@pytest.mark.parametrize("f", PAPER_FORMATS)
def test_learned_rounding_brackets(f):
    g, cm = _grid(f)
    sg = np.concatenate([-g[::-1], g[1:]])  # signed grid, ascending, single zero
    tab = O.decode_table(f)
    for t in _sweep_points(f):
        a = min(max(float(t), -cm), cm)
        q0 = tab[O.quantize_one(t, 1.0, f, 0)]
        q1 = tab[O.quantize_one(t, 1.0, f, 1)]
        lo = sg[sg <= a].max()
        assert q0 == lo, (f, t, q0, lo)          # h = 0: largest grid value not above a
        neg_pow2 = a < 0 and np.log2(-a) == np.floor(np.log2(-a)) and -a > 2.0 ** (1 - f.B)
        if neg_pow2:
            # the step of the input's binade is twice the grid spacing just above it
            step = 2.0 ** (np.log2(-a) - f.m)
            assert q1 == a + step
        elif lo == cm:
            assert q1 == cm                       # clamp
        else:
            assert q1 == sg[sg > lo].min(), (f, t, q1)   # h = 1: the grid successor
        r = tab[O.quantize_one(t, 1.0, f, -1)]
        assert r in (q0, q1)


def test_hand_worked_e2m1_cases():
    tab = O.decode_table(O.E2M1)
    modes = {"rtn": -1, "h0": 0, "h1": 1}
    n = 0
    for mode, x, want in _rows("e2m1_cases.txt"):
        code = O.quantize_one(float(x), 1.0, O.E2M1, modes[mode])
        assert tab[code] == float(want), (mode, x, tab[code], want)
        if float(want) == 0:
            assert code == 0      # zero is always +0
        n += 1
    assert n > 40


# ---- library special cases ------------------------------------------------------

def test_e4m3_rtn_equals_torch_cast_in_range():
    rng = np.random.default_rng(7)
    x = np.concatenate([rng.standard_normal(200000) * 50, rng.standard_normal(50000) * 0.01,
                        rng.uniform(-448, 448, 50000)]).astype(np.float32)
    x = x[np.abs(x) <= 448]
    got = O.quantize_act(x, 1.0, O.E4M3)
    want = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy().copy()
    want[want == 0x80] = 0
    assert np.array_equal(got, want)


def test_e5m2_rtn_equals_torch_cast_in_range():
    rng = np.random.default_rng(8)
    x = np.concatenate([rng.standard_normal(100000) * 3000, rng.standard_normal(50000) * 1e-4]).astype(np.float32)
    x = x[np.abs(x) <= 57344]
    got = O.quantize_act(x, 1.0, O.E5M2)
    want = torch.from_numpy(x).to(torch.float8_e5m2).view(torch.uint8).numpy().copy()
    want[want == 0x80] = 0
    assert np.array_equal(got, want)


def test_e1m2_is_the_uniform_integer_quantizer():
    # Uniform grid, step s = 1/4, symmetric range: s * clamp(round(x / s), -7, 7)
    rng = np.random.default_rng(9)
    x = (rng.standard_normal(20000) * 1.2).astype(np.float32)
    codes = np.array([O.quantize_one(v, 1.0, O.E1M2, -1) for v in x[:4000]])
    got = O.decode_table(O.E1M2)[codes]
    want = 0.25 * np.clip(np.rint(x[:4000].astype(np.float64) / 0.25), -7, 7)
    assert np.array_equal(got, want)


# ---- invariants on random data ---------------------------------------------------

@pytest.mark.parametrize("f", [O.E4M3, O.E2M1, O.E2M5, O.Format(5, 2, 15, 0)])
def test_invariants_random(f):
    rng = np.random.default_rng(11)
    scale = np.float32(0.0371)
    x = np.sort((rng.standard_normal(30000) * scale * O.cmax(f) / 3).astype(np.float32))
    tab = O.decode_table(f)
    w = x.reshape(1, -1)
    sc = np.array([scale], dtype=np.float32)
    unpack = (lambda c: c) if f.bits == 8 else (lambda c: np.stack([c & 15, c >> 4], -1).reshape(1, -1)[:, : x.size])
    qr = tab[unpack(O.quantize_weight(w, sc, f))][0]
    q0 = tab[unpack(O.quantize_weight(w, sc, f, O.pack_bits(np.zeros_like(w, dtype=np.uint8))))][0]
    q1 = tab[unpack(O.quantize_weight(w, sc, f, O.pack_bits(np.ones_like(w, dtype=np.uint8))))][0]
    assert np.all(np.diff(qr) >= 0) and np.all(np.diff(q0) >= 0)          # monotone
    t = (x * (np.float32(1.0) / scale)).astype(np.float32).astype(np.float64)
    cm = O.cmax(f)
    a = np.clip(t, -cm, cm)
    fl = np.floor(np.log2(np.maximum(np.abs(a), 1e-300)))
    s = np.where(fl + f.B < 1, 2.0 ** (1 - f.B - f.m), 2.0 ** (fl - f.m))
    assert np.all(np.abs(a - qr) <= s / 2)                                 # nearest
    inr = np.abs(a) < cm
    assert np.all(q0[inr] <= a[inr]) and np.all(a[inr] < q1[inr])         # bracket
    assert np.all((qr == q0) | (qr == q1))


def test_bias_and_scale_are_one_degree_of_freedom():
    rng = np.random.default_rng(12)
    x = (rng.standard_normal(5000) * 3).astype(np.float32)
    base = O.quantize_act(x, 0.05, O.Format(4, 3, 7, 0))
    for j in (-2, 1, 3):
        other = O.quantize_act(x, np.float32(0.05) * np.float32(2.0 ** -j), O.Format(4, 3, 7 - j, 0))
        assert np.array_equal(base, other)


def test_special_inputs():
    for f in (O.E4M3, O.E2M1):
        top = (1 << (f.e + f.m)) - 1 if f.sat == O.SAT_PAPER else 0x7E
        assert O.quantize_one(np.inf, 1.0, f) == top
        assert O.quantize_one(-np.inf, 1.0, f) == top | (1 << (f.e + f.m))
        assert O.quantize_one(np.nan, 1.0, f) == 0
        assert O.quantize_one(-0.0, 1.0, f) == 0
        assert O.quantize_one(-1e-30, 1.0, f) == 0          # rounds to zero: +0
        assert O.quantize_one(-1e-30, 1.0, f, 1) == 0        # floor = -1 step, +1 -> 0


def test_nibble_and_bit_packing():
    w = np.array([[0.5, -1.0, 6.0], [3.0, 0.0, -0.5]], dtype=np.float32)
    c = O.quantize_weight(w, np.ones(2, np.float32), O.E2M1)
    assert c.shape == (2, 2)
    assert list(c[0]) == [0x1 | (0xA << 4), 0x7] and list(c[1]) == [0x5 | (0x0 << 4), 0x9]
    bits = np.zeros((1, 10), dtype=np.uint8)
    bits[0, 1] = 1
    bits[0, 9] = 1
    assert list(O.pack_bits(bits)[0]) == [0x02, 0x02]
    ww = np.full((1, 10), 2.5, dtype=np.float32)
    cc = O.quantize_weight(ww, np.ones(1, np.float32), O.E4M3, O.pack_bits(bits))
    tab = O.decode_table(O.E4M3)
    # the formula adds a whole step where h = 1 even for a value already on the grid
    assert list(tab[cc[0]]) == [2.5, 2.75, 2.5, 2.5, 2.5, 2.5, 2.5, 2.5, 2.5, 2.75]
    ww[:] = 2.6
    cc = O.quantize_weight(ww, np.ones(1, np.float32), O.E4M3, O.pack_bits(bits))
    assert list(tab[cc[0]]) == [2.5, 2.75, 2.5, 2.5, 2.5, 2.5, 2.5, 2.5, 2.5, 2.75]


# ---- the layer ----------------------------------------------------------------------

def _torch_decode_e4m3(codes):
    return torch.from_numpy(np.ascontiguousarray(codes)).view(torch.float8_e4m3fn).double().numpy()


E2M1_VALUES = np.array([0, 0.5, 1, 1.5, 2, 3, 4, 6, 0, -0.5, -1, -1.5, -2, -3, -4, -6], dtype=np.float64)


def test_linear_equals_numpy_float64_matmul():
    rng = np.random.default_rng(21)
    M, N, K = 37, 29, 83
    xc = rng.integers(0, 256, (M, K)).astype(np.uint8)
    xc[(xc & 0x7F) == 0x7F] = 0
    wc8 = rng.integers(0, 256, (N, K)).astype(np.uint8)
    wc8[(wc8 & 0x7F) == 0x7F] = 0
    ws = rng.uniform(0.001, 0.01, N).astype(np.float32)
    bias = rng.standard_normal(N).astype(np.float32)
    y, ab = O.linear_codes(xc, wc8, ws, 0.013, O.E4M3, O.E4M3, bias, M, N, K)
    X = _torch_decode_e4m3(xc)
    Wd = _torch_decode_e4m3(wc8)
    g = np.float64(np.float32(0.013)) * ws.astype(np.float64)
    want = (X @ Wd.T) * g + bias
    assert np.allclose(y, want, rtol=1e-12, atol=1e-12)
    assert np.allclose(ab, (np.abs(X) @ np.abs(Wd).T) * g, rtol=1e-12)
    # 4-bit weights, packed nibbles, odd K
    wn = rng.integers(0, 16, (N, K)).astype(np.uint8)
    packed = np.zeros((N, (K + 1) // 2), np.uint8)
    packed[:, : K // 2] = wn[:, 0:K - 1:2] | (wn[:, 1::2] << 4)
    packed[:, -1] = wn[:, K - 1]
    y4, _ = O.linear_codes(xc, packed, ws, 0.013, O.E4M3, O.E2M1, None, M, N, K)
    want4 = (X @ E2M1_VALUES[wn].T) * g
    assert np.allclose(y4, want4, rtol=1e-12, atol=1e-12)
    # sampled evaluation returns the same numbers
    idx = np.array([0, 5, M * N - 1, 17 * N + 3])
    ys, _ = O.linear_codes(xc, wc8, ws, 0.013, O.E4M3, O.E4M3, bias, M, N, K, idx=idx)
    assert np.array_equal(ys, y.reshape(-1)[idx])


def test_linear_small_integers_exact():
    rng = np.random.default_rng(22)
    M, N, K = 8, 8, 64
    ints = np.array([0, 1, 2, -1, -2], dtype=np.float32)
    x = ints[rng.integers(0, 5, (M, K))]
    w = ints[rng.integers(0, 5, (N, K))]
    y, _ = O.linear(x, w, np.ones(N, np.float32), 1.0, O.E4M3, O.E4M3)
    assert np.array_equal(y, x.astype(np.float64) @ w.astype(np.float64).T)
    y, _ = O.linear(x * 4, w * 0.5, np.full(N, 0.5, np.float32), 4.0, O.E4M3, O.E2M1)
    assert np.array_equal(y, 2.0 * (x.astype(np.float64) @ w.astype(np.float64).T))


@pytest.mark.parametrize("R,pad,stride", [(3, 1, 1), (3, 1, 2), (1, 0, 1), (3, 0, 1)])
def test_conv_equals_torch_float64_conv(R, pad, stride):
    rng = np.random.default_rng(23)
    B, C, H, W, Co = 2, 5, 9, 8, 6
    xc = rng.integers(0, 256, (B, C, H, W)).astype(np.uint8)
    xc[(xc & 0x7F) == 0x7F] = 0
    wc = rng.integers(0, 256, (Co, C * R * R)).astype(np.uint8)
    wc[(wc & 0x7F) == 0x7F] = 0
    ws = rng.uniform(0.001, 0.01, Co).astype(np.float32)
    bias = rng.standard_normal(Co).astype(np.float32)
    y, ab = O.conv2d_codes(xc, wc, ws, 0.5, O.E4M3, O.E4M3, bias, B, C, H, W, Co, R, R, pad, stride)
    X = torch.from_numpy(_torch_decode_e4m3(xc))
    Wd = torch.from_numpy(_torch_decode_e4m3(wc)).reshape(Co, C, R, R)
    want = torch.nn.functional.conv2d(X, Wd, None, stride=stride, padding=pad).numpy()
    want = want * (0.5 * ws.astype(np.float64)).reshape(1, -1, 1, 1) + bias.reshape(1, -1, 1, 1)
    assert y.shape == want.shape
    assert np.allclose(y, want, rtol=1e-12, atol=1e-12)
    idx = np.array([0, 7, y.size - 1])
    ys, _ = O.conv2d_codes(xc, wc, ws, 0.5, O.E4M3, O.E4M3, bias, B, C, H, W, Co, R, R, pad, stride, idx=idx)
    assert np.array_equal(ys, y.reshape(-1)[idx])


def test_conv_1x1_is_linear_and_one_hot_tap_is_a_shift():
    rng = np.random.default_rng(24)
    B, C, H, W, Co = 2, 7, 6, 5, 4
    x = rng.standard_normal((B, C, H, W)).astype(np.float32)
    w = (rng.standard_normal((Co, C, 1, 1)) * 0.1).astype(np.float32)
    ws = np.full(Co, 0.01, np.float32)
    yc, _ = O.conv2d(x, w, ws, 0.02, O.E4M3, O.E4M3)
    yl, _ = O.linear(x.transpose(0, 2, 3, 1).reshape(-1, C), w.reshape(Co, C), ws, 0.02, O.E4M3, O.E4M3)
    assert np.array_equal(yc.transpose(0, 2, 3, 1).reshape(-1, Co), yl)
    # one-hot 3x3 kernel at tap (r, s): output is the dequantized input shifted by (r-1, s-1)
    xq = O.decode_table(O.E4M3)[O.quantize_act(x, 0.02, O.E4M3)] * np.float64(np.float32(0.02))
    for r, s in [(0, 0), (1, 2), (2, 1)]:
        w3 = np.zeros((1, C, 3, 3), np.float32)
        w3[0, 2, r, s] = 1.0
        y, _ = O.conv2d(x, w3, np.ones(1, np.float32), 0.02, O.E4M3, O.E4M3, pad=1)
        want = np.zeros((B, H, W))
        for oy in range(H):
            for ox in range(W):
                iy, ix = oy + r - 1, ox + s - 1
                if 0 <= iy < H and 0 <= ix < W:
                    want[:, oy, ox] = xq[:, 2, iy, ix]
        assert np.array_equal(y[:, 0], want)
