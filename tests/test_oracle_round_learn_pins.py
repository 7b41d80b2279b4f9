"""Pins of the oracle's rounding-learning step (Sec. V-B) against things it does not compute itself:
closed forms of the regulariser, the hardened quantizer as the limit of the soft one, a brute-force
neighbour search over the decoded grid differentiated by autograd, and central differences of the
objective."""
import math

import numpy as np
import pytest
import torch

import oracle as O

FORMATS = [O.E2M1, O.E1M2, O.Format(2, 1, 2, O.SAT_PAPER), O.E3M4]


def _case(f, seed, N=6, K=24, M=40):
    rng = np.random.default_rng(seed)
    w = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    w[0, 0] = 0.0
    scale = np.array([O.scale_from_max(v, f) for v in np.abs(w).max(axis=1)], dtype=np.float32)
    scale[1] *= np.float32(0.6)                           # one row whose largest weights are clipped
    # alpha on a coarse binary grid so that alpha +- h is exact in FP32
    alpha = (np.round(rng.standard_normal((N, K)) * 2.0 * 64) / 64).astype(np.float32)
    a = rng.standard_normal((M, K)).astype(np.float32)
    return w, scale, alpha, a


def test_regulariser_closed_forms():
    al = np.array([0.0, math.log(3.0), -math.log(3.0), 50.0, -50.0], dtype=np.float64)
    lam, dlam = O.rounding_regularizer(al)
    assert lam[0] == 1.0                                   # sigma = 0.5: undecided, largest penalty
    assert lam[1] == pytest.approx(1.0 - 0.5 ** 20, rel=1e-14)   # sigma = 0.75
    assert lam[2] == pytest.approx(lam[1], rel=1e-14)     # even in alpha
    assert abs(lam[3]) < 1e-15 and abs(lam[4]) < 1e-15    # decided: no penalty
    assert dlam[0] == 0.0
    # sigma = 0.75: d lambda / d alpha = -20 * 0.5^19 * 2 * sigma (1 - sigma)
    assert dlam[1] == pytest.approx(-20 * 0.5 ** 19 * 2 * 0.75 * 0.25, rel=1e-12)
    assert dlam[2] == pytest.approx(-dlam[1], rel=1e-12)
    # derivative against central differences
    x = np.linspace(-6, 6, 49)
    h = 1e-6
    num = (O.rounding_regularizer(x + h)[0] - O.rounding_regularizer(x - h)[0]) / (2 * h)
    np.testing.assert_allclose(O.rounding_regularizer(x)[1], num, rtol=1e-6, atol=1e-9)


@pytest.mark.parametrize("f", FORMATS)
def test_saturated_alpha_gives_the_hardened_quantizer(f):
    # sigma(-800) = 0 and sigma(800) = 1 exactly: the soft weights are the floor + bit quantizer
    w, scale, _, _ = _case(f, 1)
    rng = np.random.default_rng(2)
    bits = rng.integers(0, 2, size=w.shape).astype(np.uint8)
    alpha = np.where(bits == 1, 800.0, -800.0).astype(np.float32)
    with np.errstate(over="ignore"):
        wq, dwq = O.soft_weight(w, scale, f, alpha)
    codes = O.quantize_weight(w, scale, f, O.pack_bits(bits))
    table = O.decode_table(f)
    if f.bits == 4:
        lo, hi = codes & 0xF, codes >> 4
        flat = np.stack([lo, hi], axis=-1).reshape(w.shape[0], -1)[:, : w.shape[1]]
    else:
        flat = codes
    want = table[flat] * scale.astype(np.float64)[:, None]
    assert np.array_equal(wq, want)
    assert np.all(dwq == 0.0)                              # sigma' vanishes at both ends


@pytest.mark.parametrize("f", FORMATS)
def test_soft_weight_is_linear_between_the_two_hardened_values(f):
    w, scale, alpha, _ = _case(f, 3)
    with np.errstate(over="ignore"):
        lo, _ = O.soft_weight(w, scale, f, np.full_like(alpha, -800.0))
    wq, _ = O.soft_weight(w, scale, f, alpha)
    sig = 1.0 / (1.0 + np.exp(-alpha.astype(np.float64)))
    # step from the brute-force neighbour search: distance from lo to the next grid value above it
    table = np.unique(O.decode_table(f))
    c = O.cmax(f)
    for n in range(w.shape[0]):
        for k in range(w.shape[1]):
            g = lo[n, k] / float(scale[n])
            above = table[table > g + 1e-12]
            t = float(np.float32(w[n, k]) * (np.float32(1.0) / scale[n]))
            negative_power_of_two = t < 0 and math.log2(-t) == math.floor(math.log2(-t))
            if above.size == 0 or negative_power_of_two:
                continue
            step = above[0] - g
            want = float(scale[n]) * min(g + step * sig[n, k], c)
            assert wq[n, k] == pytest.approx(want, rel=1e-13, abs=1e-18)


def test_weights_on_the_grid_with_round_down_give_zero_loss():
    f = O.E2M1
    rng = np.random.default_rng(4)
    table = O.decode_table(f)
    w = (table[rng.integers(0, 16, size=(5, 16))] * 0.25).astype(np.float32)
    scale = np.full(5, 0.25, dtype=np.float32)
    a = rng.standard_normal((12, 16)).astype(np.float32)
    with np.errstate(over="ignore"):
        mse, reg = O.round_learn_loss(w, scale, f, np.full_like(w, -800.0), a, 0.0)
    assert mse == 0.0 and reg == 0.0


@pytest.mark.parametrize("f", FORMATS)
def test_gradient_matches_central_differences_of_the_objective(f):
    w, scale, alpha, a = _case(f, 5)
    reg = 0.01
    r = O.round_learn_step(w, scale, f, alpha, a, reg)
    h = np.float32(2.0 ** -12)
    rng = np.random.default_rng(6)
    picks = [(0, 0)] + [(int(rng.integers(0, w.shape[0])), int(rng.integers(0, w.shape[1]))) for _ in range(30)]
    picks += [(1, int(k)) for k in np.argsort(-np.abs(w[1]))[:3]]          # clipped weights
    for n, k in picks:
        ap, am = alpha.copy(), alpha.copy()
        ap[n, k] += h
        am[n, k] -= h
        lp = O.round_learn_loss(w, scale, f, ap, a, reg)
        lm = O.round_learn_loss(w, scale, f, am, a, reg)
        num = ((lp[0] + reg * lp[1]) - (lm[0] + reg * lm[1])) / (2.0 * float(h))
        assert r["grad"][n, k] == pytest.approx(num, rel=2e-5, abs=1e-11), (n, k)


def test_gradient_matches_autograd_through_a_grid_neighbour_search():
    # E2M1: the grid written out; lower neighbour by search, upper neighbour its successor.
    f = O.E2M1
    w, scale, alpha, a = _case(f, 7)
    grid = torch.tensor([-6, -4, -3, -2, -1.5, -1, -0.5, 0, 0.5, 1, 1.5, 2, 3, 4, 6], dtype=torch.float64)
    t = torch.from_numpy(w * (np.float32(1.0) / scale)[:, None]).to(torch.float64)
    t = t.clamp(-6.0, 6.0)
    below = (grid[None, None, :] <= t[..., None])
    lo_idx = below.to(torch.int64).sum(-1) - 1
    lo = grid[lo_idx]
    hi = grid[torch.clamp(lo_idx + 1, max=grid.numel() - 1)]
    step = torch.where(hi > lo, hi - lo, torch.tensor(2.0, dtype=torch.float64))   # above 6: step of the top binade
    al = torch.from_numpy(alpha).to(torch.float64).requires_grad_(True)
    sc = torch.from_numpy(scale).to(torch.float64)[:, None]
    wq = sc * torch.clamp(lo + step * torch.sigmoid(al), -6.0, 6.0)
    A = torch.from_numpy(a).to(torch.float64)
    W = torch.from_numpy(w).to(torch.float64)
    reg = 0.02
    lam = 1.0 - (2.0 * (torch.sigmoid(al) - 0.5).abs()) ** 20
    loss = ((A @ wq.T - A @ W.T) ** 2).mean() + reg * lam.sum()
    loss.backward()
    r = O.round_learn_step(w, scale, f, alpha, a, reg)
    assert r["mse"] + reg * r["reg"] == pytest.approx(float(loss.detach()), rel=1e-12)
    np.testing.assert_allclose(r["grad"], al.grad.numpy(), rtol=1e-10, atol=1e-16)
    np.testing.assert_allclose(r["wq"], wq.detach().numpy(), rtol=1e-14, atol=0)


@pytest.mark.parametrize("shape", [(2, 3, 7, 6, 3, 3, 1, 1), (1, 4, 8, 8, 3, 3, 1, 2), (2, 5, 5, 9, 1, 1, 0, 1), (1, 2, 6, 6, 3, 2, 0, 1)])
def test_unfold_is_the_library_unfold_and_turns_the_convolution_into_a_product(shape):
    B, C, H, W, R, S, pad, stride = shape
    rng = np.random.default_rng(sum(shape))
    x = rng.standard_normal((B, C, H, W)).astype(np.float32)
    rows = O.unfold(x, R, S, pad, stride)
    lib = torch.nn.functional.unfold(torch.from_numpy(x), (R, S), padding=pad, stride=stride)   # [B][C*R*S][L]
    assert np.array_equal(rows, lib.permute(0, 2, 1).reshape(rows.shape).numpy())
    # rows times flattened weights = the convolution
    w = rng.standard_normal((4, C, R, S)).astype(np.float32)
    y = torch.nn.functional.conv2d(torch.from_numpy(x).double(), torch.from_numpy(w).double(), padding=pad, stride=stride)
    got = rows.astype(np.float64) @ w.reshape(4, -1).astype(np.float64).T
    np.testing.assert_allclose(got, y.permute(0, 2, 3, 1).reshape(got.shape).numpy(), rtol=1e-12, atol=1e-12)
