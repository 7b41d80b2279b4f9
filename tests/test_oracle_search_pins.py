"""Pins of the oracle's encoding / bias search (Sec. V-A, Algorithm 1) against things it does not
compute itself: library casts, a uniform-grid closed form, brute force over the decoded grid, and
hand-made error tables for the selection rule."""
import numpy as np
import pytest
import torch

import oracle as O


def _brute_force_mse(x, f, c):
    """Nearest grid point by exhaustive search over the decoded codes (ties to the even code)."""
    table = O.decode_table(f)
    half = table[: table.size // 2]                      # non-negative codes, increasing
    scale = np.float32(np.float32(c) / np.float32(O.cmax(f)))
    r = np.float32(1.0) / scale
    total = 0.0
    for v in x:
        t = float(np.float32(v) * r)
        a = min(abs(t), O.cmax(f))
        d = np.abs(half - a)
        best = np.flatnonzero(d == d.min())
        code = best[0] if best.size == 1 or best[0] % 2 == 0 else best[1]
        q = np.sign(t) * half[code]
        total += (float(v) - float(scale) * q) ** 2
    return total / len(x)


@pytest.mark.parametrize("f", [O.E2M1, O.E1M2, O.E3M4, O.E2M5, O.Format(4, 3, 8, O.SAT_PAPER),
                               O.Format(5, 2, 16, O.SAT_PAPER)])
def test_mse_is_the_brute_force_nearest_grid_point_error(f):
    rng = np.random.default_rng(5)
    x = (rng.standard_normal(300) * 1.3).astype(np.float32)
    x[:4] = [0.0, -0.0, 7.5, -9.0]                       # zeros and values that get clipped
    clips = np.array([0.37, 1.0, 2.9, 5.0], dtype=np.float32)
    got = O.search_mse(x, [f], clips)[0]
    want = [_brute_force_mse(x, f, c) for c in clips]
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=0)


def test_e4m3_matches_the_library_cast_in_range():
    # power-of-two scale: t = x / scale is exact, and below 448 the paper's E4M3 grid (bias 7) is
    # the one of torch.float8_e4m3fn
    f = O.Format(4, 3, 7, O.SAT_PAPER)
    rng = np.random.default_rng(6)
    for k in (-3, 0, 4):
        scale = 2.0 ** k
        x = (rng.standard_normal(5000) * 100 * scale).astype(np.float32)
        x = x[np.abs(x) <= 448 * scale]
        xq = torch.from_numpy(x / np.float32(scale)).to(torch.float8_e4m3fn).to(torch.float64).numpy() * scale
        want = np.mean((x.astype(np.float64) - xq) ** 2)
        got = O.search_mse(x, [f], [480.0 * scale])[0, 0]
        assert got == pytest.approx(want, rel=1e-12)


def test_e1m2_is_the_uniform_quantizer():
    # E1M2 with bias 1 is the uniform grid {0, 0.25, ..., 1.75}: the integer quantizer of Sec. IV-A
    rng = np.random.default_rng(7)
    x = (rng.standard_normal(4000)).astype(np.float32)
    for k in (-2, 0, 1):
        scale = 2.0 ** k
        xq = np.clip(np.round(x.astype(np.float64) / scale * 4) / 4, -1.75, 1.75) * scale
        want = np.mean((x.astype(np.float64) - xq) ** 2)
        got = O.search_mse(x, [O.E1M2], [1.75 * scale])[0, 0]
        assert got == pytest.approx(want, rel=1e-12)


def test_data_on_a_grid_has_zero_error_and_is_selected():
    f = O.Format(2, 1, 2, O.SAT_PAPER)                   # grid {0, .25, .5, .75, 1, 1.5, 2, 3}
    grid = np.array([0, .25, .5, .75, 1, 1.5, 2, 3])
    rng = np.random.default_rng(8)
    x = (rng.choice(grid, 500) * rng.choice([-1, 1], 500) * 0.5).astype(np.float32)   # scale 0.5, c = 1.5
    x[0] = 1.5
    clips = O.clip_candidates(1.5, 6)                    # 0.25 .. 1.5
    mse = O.search_mse(x, O.FP4_ENCODINGS, clips)
    assert mse[1, 5] == 0.0
    assert (np.delete(mse.reshape(-1), 1 * 6 + 5) > 0).all()
    assert O.select_encoding_and_bias(mse) == (1, 5)


def test_integer_bias_only_fixes_the_unit():
    # the same (e, m) with another integer bias and the same clipping value is the same quantizer
    rng = np.random.default_rng(9)
    x = rng.standard_normal(2000).astype(np.float32)
    clips = O.clip_candidates(np.abs(x).max(), 7)
    a = O.search_mse(x, [O.Format(3, 4, 4, O.SAT_PAPER)], clips)
    b = O.search_mse(x, [O.Format(3, 4, 2, O.SAT_PAPER)], clips)
    assert np.array_equal(a, b)


def test_clipping_value_and_bias_are_one_parameter():
    # clipping equation, both directions, at the integer biases where it can be checked by hand
    assert O.bias_from_clip(240.0, O.E4M3) == pytest.approx(8.0)
    assert O.bias_from_clip(480.0, O.E4M3) == pytest.approx(7.0)
    assert O.bias_from_clip(6.0, O.E2M1) == pytest.approx(1.0)
    assert O.bias_from_clip(3.0, O.E2M1) == pytest.approx(2.0)
    assert O.bias_from_clip(1.75, O.E1M2) == pytest.approx(1.0)
    assert O.bias_from_clip(57344.0, O.Format(5, 2, 16, 0)) == pytest.approx(16.0)
    assert O.bias_from_clip(3.0 * 2 ** 0.5, O.E2M1) == pytest.approx(1.5)     # a real-valued bias


def test_clip_candidates_are_evenly_spaced_up_to_the_maximum():
    c = O.clip_candidates(3.7)
    assert c.size == 111 and c.dtype == np.float32
    assert c[-1] == np.float32(3.7)
    assert (np.diff(c) > 0).all()
    np.testing.assert_allclose(c, float(np.float32(3.7)) * np.arange(1, 112) / 111, rtol=6e-8)


def test_selection_keeps_the_first_strict_minimum():
    mse = np.array([[5.0, 3.0, 4.0], [3.0, 2.0, 2.0], [2.0, 9.0, 2.5]])
    assert O.select_encoding_and_bias(mse) == (1, 1)     # later equal values do not replace it
    assert O.select_encoding_and_bias(np.array([[1.0]])) == (0, 0)    # start value is +infinity
    mse[1, 1] = np.nan                                    # a NaN error is never selected
    assert O.select_encoding_and_bias(mse) == (1, 2)


def test_selection_with_tied_minima_takes_the_first_in_encoding_major_order():
    # ties inside a row, across rows, at the very first entry, and an all-infinite table
    assert O.select_encoding_and_bias(np.array([[1.0, 1.0], [1.0, 1.0]])) == (0, 0)
    assert O.select_encoding_and_bias(np.array([[4.0, 2.0, 2.0], [2.0, 7.0, 2.0]])) == (0, 1)
    assert O.select_encoding_and_bias(np.array([[np.inf, 3.0], [3.0, 3.0]])) == (0, 1)
    assert O.select_encoding_and_bias(np.array([[np.nan, 6.0], [5.0, 5.0]])) == (1, 0)
    assert O.select_encoding_and_bias(np.full((2, 3), np.inf)) == (None, None)
    assert O.select_encoding_and_bias(np.full((2, 3), np.nan)) == (None, None)
    # against the definition spelled out: smallest value, then smallest encoding index, then smallest candidate index
    rng = np.random.default_rng(5)
    for _ in range(200):
        t = rng.integers(0, 4, size=(4, 7)).astype(np.float64)          # few distinct values: many ties
        t[rng.random(t.shape) < 0.1] = np.nan
        finite = [(t[i, j], i, j) for i in range(4) for j in range(7) if not np.isnan(t[i, j])]
        want = min(finite)[1:] if finite else (None, None)
        assert O.select_encoding_and_bias(t) == want


def test_narrow_data_takes_the_most_mantissa_bits_and_heavy_tails_take_fewer():
    rng = np.random.default_rng(10)
    narrow = rng.uniform(-1, 1, 20000).astype(np.float32)
    i, _ = O.select_encoding_and_bias(O.search_mse(narrow, O.FP8_ENCODINGS, O.clip_candidates(1.0, 16)))
    assert O.FP8_ENCODINGS[i].m == 5
    heavy = (rng.standard_normal(20000) * np.exp(3 * rng.standard_normal(20000))).astype(np.float32)
    i, _ = O.select_encoding_and_bias(O.search_mse(heavy, O.FP8_ENCODINGS,
                                                   O.clip_candidates(np.abs(heavy).max(), 16)))
    assert O.FP8_ENCODINGS[i].m < 5


def test_zero_count_is_the_number_of_values_that_decode_to_zero():
    rng = np.random.default_rng(11)
    for f in (O.E4M3, O.E2M1, O.E1M2, O.E3M4):
        for n in (1, 2, 7, 1000, 1001):
            x = (rng.standard_normal(n) * 0.3).astype(np.float32)
            x[rng.random(n) < 0.2] = 0.0
            codes = O.quantize_act(x, 0.5, f)
            table = O.decode_table(f)
            decoded = np.array([table[O.quantize_one(v, 0.5, f)] for v in x])
            assert O.zero_count(codes, n, f) == int(np.count_nonzero(decoded == 0.0))
    assert O.zero_count(np.array([0x10, 0x00, 0x0F], dtype=np.uint8), 5, O.E2M1) == 3   # 0,1 | 0,0 | f,(pad)
    assert O.zero_count(np.array([0x10, 0x00, 0x0F], dtype=np.uint8), 6, O.E2M1) == 4
    assert O.zero_count(np.array([0, 0x80, 3, 0], dtype=np.uint8), 4, O.E4M3) == 2      # 0x80 would be -0: not produced, not counted
