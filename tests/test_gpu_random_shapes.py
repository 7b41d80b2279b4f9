"""Seeded random conv / linear shapes through both routes of the library against the oracle: a net
under the hand-picked cases, cast over the kernel's many plans (row / framed / per-tap addressing,
resident or streamed operands, cluster split, paired row tiles, few-row path, ragged everything)."""
import numpy as np
import pytest

from paper_2408_06995_b200 import inputs as I
from _helpers import layer_scales, gpu_layer, oracle_layer, assert_close, sample_indices

pytestmark = pytest.mark.gpu


def _random_layer(rng, j):
    pick = lambda a: int(rng.choice(a))
    wfmt = ["e4m3", "e2m1"][pick([0, 1])]
    rounding = bool(rng.random() < 0.5)
    if rng.random() < 0.35:
        M = pick([1, 2, 3, 7, 8, 9, 64, 127, 128, 129, 154, 300, 512, 1000, 2048])
        K = pick([16, 48, 100, 128, 130, 320, 640, 768, 1000, 1280, 2560, 4100])
        N = pick([1, 4, 40, 64, 65, 128, 200, 320, 640, 1000, 1280])
        return I.linear_layer(f"r{j}", M, K, N, wfmt, rounding=rounding)
    while True:
        R = pick([1, 3, 3, 3])
        stride = pick([1, 1, 1, 2])
        pad = R // 2 if rng.random() < 0.85 else 0
        H = pick([4, 7, 8, 9, 16, 17, 32, 33, 64])
        W = H if rng.random() < 0.7 else pick([5, 8, 13, 32])
        B = pick([1, 2, 3, 5, 17])
        C = pick([3, 4, 16, 20, 64, 128, 130, 256, 320, 640, 960, 1280])
        Co = pick([1, 4, 24, 64, 100, 128, 200, 320, 640])
        if H + 2 * pad < R or W + 2 * pad < R or B * C * H * W > 4e6 or Co * C * R * R > 6e6:
            continue
        return I.conv_layer(f"r{j}", B, C, H, W, Co, R, pad=pad, stride=stride, wfmt=wfmt, rounding=rounding)


@pytest.mark.parametrize("seed", range(6))
def test_random_layers_match_the_oracle(seed):
    rng = np.random.default_rng(1000 + seed)
    for j in range(25):
        L = _random_layer(rng, j)
        I.draw(L, 80 + seed, 10 * j, ["normal", "silu", "t4"][j % 3], 0.03, True)
        ws, xs = layer_scales(L)
        y = gpu_layer(L, ws, xs)                        # both routes, asserted equal
        idx = sample_indices(y.size, min(y.size, 400), j, [0, y.size - 1])
        yr, ab = oracle_layer(L, ws, xs, idx)
        assert np.all(np.isfinite(y)), (seed, j, L.name)
        assert_close(y.reshape(-1)[idx], yr, ab)
