"""GPU parity of the rounding-learning step (Sec. V-B) against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2408_06995_b200 as fpq

pytestmark = pytest.mark.gpu

# The kernels work in FP32 (the method's own precision), the oracle in double.  Every term of the two
# contractions is rounded once and summed in FP32: |err| <= (terms * 2^-24) * sum |terms|, at most 1e-3 of the
# sum of absolute terms for reductions of up to 16384 elements (typical errors are sqrt(terms) smaller).  The
# gradient bound below also carries the error of its left operand D = A (Wq - W)^T, which has the same form.
# The regulariser's derivative is a product of a few FP32 library results (exp, tanh, a 19th power by repeated
# squaring): a relative error below 1e-5.  The oracle forms 1 - sigma and sigma - 0.5 by subtraction in double, an
# absolute error of 2^-53 that the factor 40 u^19 <= 40 carries into the derivative: 1e-14 * reg covers it.
GRAD_RTOL_ABSUM = 1e-3
LOSS_RTOL = 2e-5

PAIRS = [(fpq.E2M1, O.E2M1), (fpq.E1M2, O.E1M2), (fpq.E3M4, O.E3M4), (fpq.E4M3, O.E4M3)]


def _case(M, N, K, ofmt, seed):
    rng = np.random.default_rng(seed)
    w = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    scale = np.array([O.scale_from_max(v, ofmt) for v in np.abs(w).max(axis=1) + 1e-12], dtype=np.float32)
    if N > 1:
        scale[1] *= np.float32(0.6)                      # a row whose largest weights are clipped
    alpha = (rng.standard_normal((N, K)) * 2.0).astype(np.float32)
    alpha.reshape(-1)[:: 17] = 0.0                       # undecided
    alpha.reshape(-1)[3:: 29] = 30.0                     # decided
    alpha.reshape(-1)[5:: 31] = -30.0
    a = rng.standard_normal((M, K)).astype(np.float32)
    a[rng.random((M, K)) < 0.0005] *= 30.0
    return w, scale, alpha, a


def _check(M, N, K, gfmt, ofmt, seed, reg=0.01, lr=0.0):
    w, scale, alpha, a = _case(M, N, K, ofmt, seed)
    d = "cuda"
    al_dev = torch.from_numpy(alpha.copy()).to(d)
    grad, loss = fpq.fpq_round_learn_step(torch.from_numpy(w).to(d), torch.from_numpy(scale).to(d), gfmt, al_dev,
                                          torch.from_numpy(a).to(d), reg, lr)
    assert fpq.fpq_read_status() == fpq.OK
    r = O.round_learn_step(w, scale, ofmt, alpha, a, reg)
    g = grad.cpu().numpy().astype(np.float64)
    ls = loss.cpu().numpy()
    assert ls[0] == pytest.approx(r["mse"], rel=LOSS_RTOL, abs=1e-30)
    assert ls[1] == pytest.approx(r["reg"], rel=LOSS_RTOL, abs=1e-6)
    # second-level bound: the error of D enters the gradient through sum_m |dD| |A|
    absum_d = np.abs(a.astype(np.float64)) @ np.abs(r["wq"] - w.astype(np.float64)).T
    dwq = np.abs(O.soft_weight(w, scale, ofmt, alpha)[1])
    second = (2.0 / (M * N)) * (absum_d.T @ np.abs(a.astype(np.float64))) * dwq
    tol = GRAD_RTOL_ABSUM * (r["absum"] + second) + 4.0 * np.spacing(np.abs(r["grad"]).astype(np.float32)).astype(np.float64) \
        + 1e-5 * reg * np.abs(O.rounding_regularizer(alpha)[1]) + 1e-14 * reg
    err = np.abs(g - r["grad"])
    worst = np.unravel_index(np.argmax(err - tol), err.shape)
    assert np.all(err <= tol), (worst, g[worst], r["grad"][worst], err[worst], tol[worst])
    if lr != 0.0:
        want = alpha.astype(np.float64) - lr * g
        np.testing.assert_allclose(al_dev.cpu().numpy(), want, rtol=3e-7, atol=1e-7)
    else:
        assert np.array_equal(al_dev.cpu().numpy(), alpha)
    return float((err / tol).max())


@pytest.mark.parametrize("gfmt,ofmt", PAIRS)
@pytest.mark.parametrize("shape", [(300, 200, 136), (257, 129, 20), (70, 33, 27), (1, 1, 1), (513, 4, 36), (2, 260, 516)])
def test_round_learn_step_matches_the_oracle(shape, gfmt, ofmt):
    M, N, K = shape
    _check(M, N, K, gfmt, ofmt, seed=M + 3 * N + 7 * K)


def test_round_learn_descent_update():
    _check(384, 96, 160, fpq.E2M1, O.E2M1, seed=11, reg=0.02, lr=50.0)


@pytest.mark.parametrize("shape", [(4096, 320, 1280), (4096, 960, 320), (256, 1280, 5120)])
def test_round_learn_step_at_transformer_block_sizes(shape):
    # FFN-out and QKV projections of the SD-v1 style transformer block (one 64 x 64 latent of calibration rows) and
    # the deepest FFN-out (16 x 16 latent: few output tiles, sliced reduction); sizes bench.py --suite round_learn times
    M, N, K = shape
    _check(M, N, K, fpq.E2M1, O.E2M1, seed=5)


def test_tensor_core_contractions_keep_fp32_accuracy():
    """Rows of a multiple of 4 floats take the tensor cores (three TF32 products per FP32 product, the reduction
    accumulated in chunks): the result must stay at FP32 accuracy, far inside the bounds above.  A two-product
    split, an operand read with other than its leading TF32 bits, or one long truncating accumulation would show
    here as errors of 1e-4 and more."""
    for (M, N, K) in [(512, 256, 1280), (1024, 320, 5120), (300, 130, 324)]:
        w, scale, alpha, a = _case(M, N, K, O.E2M1, 7)
        d = "cuda"
        grad, loss = fpq.fpq_round_learn_step(torch.from_numpy(w).to(d), torch.from_numpy(scale).to(d), fpq.E2M1,
                                              torch.from_numpy(alpha.copy()).to(d), torch.from_numpy(a).to(d), 0.0, 0.0)
        assert fpq.fpq_read_status() == fpq.OK
        r = O.round_learn_step(w, scale, O.E2M1, alpha, a, 0.0)
        assert loss.cpu().numpy()[0] == pytest.approx(r["mse"], rel=1e-5)
        err = np.abs(grad.cpu().numpy().astype(np.float64) - r["grad"])
        assert np.all(err <= 2e-5 * r["absum"] + 4.0 * np.spacing(np.abs(r["grad"]).astype(np.float32)).astype(np.float64) + 1e-16)
        assert np.median(err[r["absum"] > 0] / r["absum"][r["absum"] > 0]) < 2e-6


def test_two_calls_on_one_workspace_agree():
    w, scale, alpha, a = _case(500, 130, 72, O.E2M1, 9)
    d = "cuda"
    args = [torch.from_numpy(v).to(d) for v in (w, scale, alpha, a)]
    ws = torch.empty(fpq.fpq_round_learn_workspace_size(500, 130, 72), dtype=torch.uint8, device=d)
    g1, l1 = fpq.fpq_round_learn_step(args[0], args[1], fpq.E2M1, args[2], args[3], 0.01, workspace=ws)
    g1, l1 = g1.clone(), l1.clone()
    g2, l2 = fpq.fpq_round_learn_step(args[0], args[1], fpq.E2M1, args[2], args[3], 0.01, workspace=ws)
    assert torch.equal(g1, g2)                            # the slices are added in a fixed order
    assert torch.allclose(l1, l2, rtol=1e-12, atol=0)     # sums of squares meet in atomics: order may differ


@pytest.mark.parametrize("shape", [(1, 1), (3, 7), (5, 8), (33, 129), (64, 320)])
def test_harden_is_the_sign_test_in_the_quantizer_bit_layout(shape):
    N, K = shape
    rng = np.random.default_rng(N * 1000 + K)
    alpha = rng.standard_normal((N, K)).astype(np.float32)
    alpha.reshape(-1)[::5] = 0.0
    alpha.reshape(-1)[1::7] = -0.0
    bits = fpq.fpq_round_learn_harden(torch.from_numpy(alpha).cuda()).cpu().numpy()
    sig = 1.0 / (1.0 + np.exp(-alpha.astype(np.float64)))
    assert np.array_equal(bits, O.pack_bits((sig >= 0.5).astype(np.uint8)))


def test_learned_bits_feed_the_weight_encoder():
    # descent steps, hardening, then the encoder: same codes as the oracle's encoder on the same bits
    w, scale, alpha, a = _case(256, 64, 96, O.E2M1, 13)
    d = "cuda"
    wd, sd, ald, ad = [torch.from_numpy(v).to(d) for v in (w, scale, alpha.copy(), a)]
    first = None
    for _ in range(20):
        _, loss = fpq.fpq_round_learn_step(wd, sd, fpq.E2M1, ald, ad, 0.0, lr=1e6)
        first = float(loss[0]) if first is None else first
    assert float(loss[0]) < 0.5 * first                   # the layer-output error went down
    bits = fpq.fpq_round_learn_harden(ald)
    codes = fpq.fpq_quantize_weight(wd, sd, fpq.E2M1, bits)
    want = O.quantize_weight(w, scale, O.E2M1, bits.cpu().numpy())
    assert np.array_equal(codes.cpu().numpy(), want)


@pytest.mark.parametrize("shape", [(2, 3, 7, 6, 3, 3, 1, 1), (1, 4, 8, 8, 3, 3, 1, 2), (3, 130, 9, 11, 1, 1, 0, 1),
                                   (2, 40, 16, 16, 3, 3, 1, 1), (1, 2, 6, 6, 3, 2, 0, 1)])
def test_unfold_matches_the_oracle_bit_for_bit(shape):
    B, C, H, W, R, S, pad, stride = shape
    rng = np.random.default_rng(sum(shape))
    x = rng.standard_normal((B, C, H, W)).astype(np.float32)
    rows = fpq.fpq_round_learn_unfold(torch.from_numpy(x).cuda(), R, S, pad, stride)
    assert np.array_equal(rows.cpu().numpy(), O.unfold(x, R, S, pad, stride))


def test_round_learn_step_for_a_convolution():
    # 3 x 3 convolution weights [Co][C][3][3] learned against the layer's own input: unfold, then the same step
    rng = np.random.default_rng(17)
    B, C, H, W, Co = 2, 24, 12, 12, 40
    x = rng.standard_normal((B, C, H, W)).astype(np.float32)
    w = (rng.standard_normal((Co, C * 9)) * 0.03).astype(np.float32)
    scale = np.array([O.scale_from_max(v, O.E2M1) for v in np.abs(w).max(axis=1)], dtype=np.float32)
    alpha = (rng.standard_normal(w.shape) * 2).astype(np.float32)
    d = "cuda"
    rows = fpq.fpq_round_learn_unfold(torch.from_numpy(x).to(d), 3, 3, 1, 1)
    grad, loss = fpq.fpq_round_learn_step(torch.from_numpy(w).to(d), torch.from_numpy(scale).to(d), fpq.E2M1,
                                          torch.from_numpy(alpha).to(d), rows, 0.01)
    r = O.round_learn_step(w, scale, O.E2M1, alpha, O.unfold(x, 3, 3, 1, 1), 0.01)
    assert float(loss[0]) == pytest.approx(r["mse"], rel=LOSS_RTOL)
    tol = 2.0 * GRAD_RTOL_ABSUM * r["absum"] + 1e-5 * 0.01 * np.abs(O.rounding_regularizer(alpha)[1]) + 1e-16 \
        + 4.0 * np.spacing(np.abs(r["grad"]).astype(np.float32)).astype(np.float64)
    assert np.all(np.abs(grad.cpu().numpy() - r["grad"]) <= tol)


def test_nan_weight_is_reported_and_contributes_nothing():
    w, scale, alpha, a = _case(64, 20, 24, O.E2M1, 3)
    d = "cuda"
    args = [torch.from_numpy(v).to(d) for v in (w, scale, alpha, a)]
    g0, l0 = fpq.fpq_round_learn_step(args[0], args[1], fpq.E2M1, args[2], args[3], 0.0)
    assert fpq.fpq_read_status() == fpq.OK
    wn = args[0].clone()
    wn[2, 7] = float("nan")
    g1, l1 = fpq.fpq_round_learn_step(wn, args[1], fpq.E2M1, args[2], args[3], 0.0)
    assert fpq.fpq_read_status() == fpq.ERR_NAN_INPUT
    assert torch.isfinite(g1).all() and torch.isfinite(l1).all()
    assert float(g1[2, 7]) == 0.0
    # rows of other output channels do not see the NaN weight at all
    keep = [n for n in range(20) if n != 2]
    assert torch.equal(g0[keep], g1[keep])
