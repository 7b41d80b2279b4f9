"""GPU parity of the encoding / bias search (Sec. V-A, Algorithm 1) against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2408_06995_b200 as fpq

pytestmark = pytest.mark.gpu

# The kernel forms each error with one FP32 rounding (fused multiply-add) and adds 512 squared
# errors in FP32 before switching to double; the oracle works in double throughout.  Relative error
# of one term <= 2^-23, of a 512-term FP32 sum <= 9 * 2^-24 with pairwise (shuffle) addition.
RTOL = 2e-6

FP8 = [fpq.Format(f.e, f.m, f.B, fpq.SAT_PAPER) for f in O.FP8_ENCODINGS]
FP4 = [fpq.Format(f.e, f.m, f.B, fpq.SAT_PAPER) for f in O.FP4_ENCODINGS]


def _tensor(kind, n, seed):
    rng = np.random.default_rng(seed)
    if kind == "normal":
        return rng.standard_normal(n).astype(np.float32)
    if kind == "weights":
        return (rng.standard_normal(n) * 0.02).astype(np.float32)
    if kind == "heavy":
        x = rng.standard_normal(n)
        x[rng.random(n) < 0.001] *= 30
        return x.astype(np.float32)
    if kind == "silu":
        z = rng.standard_normal(n)
        return (z / (1 + np.exp(-z))).astype(np.float32)
    raise ValueError(kind)


def _run(x, encs_gpu, encs_cpu, count):
    maxabs = float(np.abs(x).max())
    clips = fpq.fpq_search_clip_candidates(maxabs, count)
    assert np.array_equal(clips.numpy(), O.clip_candidates(maxabs, count))       # bit for bit
    mse, best = fpq.fpq_search_format(torch.from_numpy(x).cuda(), encs_gpu, clips.cuda())
    assert fpq.fpq_read_status() == fpq.OK
    want = O.search_mse(x, encs_cpu, clips.numpy())
    return mse.cpu().numpy(), best.cpu().numpy(), want


@pytest.mark.parametrize("kind", ["normal", "weights", "heavy", "silu"])
@pytest.mark.parametrize("n", [1, 37, 4096, 4097, 50000])
def test_fp8_search_matches_the_oracle(kind, n):
    x = _tensor(kind, n, n + 1)
    got, best, want = _run(x, FP8, O.FP8_ENCODINGS, 111)
    np.testing.assert_allclose(got, want, rtol=RTOL, atol=0)
    # the selection: exactly Algorithm 1 applied to the kernel's own errors, and as good as the
    # oracle's choice (two candidates whose errors agree to RTOL may swap)
    assert tuple(best) == O.select_encoding_and_bias(got)
    wi, wj = O.select_encoding_and_bias(want)
    assert want[best[0], best[1]] <= want[wi, wj] * (1 + 2 * RTOL)


@pytest.mark.parametrize("kind", ["normal", "weights"])
def test_fp4_search_matches_the_oracle(kind):
    x = _tensor(kind, 30000, 3)
    got, best, want = _run(x, FP4, O.FP4_ENCODINGS, 111)
    np.testing.assert_allclose(got, want, rtol=RTOL, atol=0)
    assert tuple(best) == O.select_encoding_and_bias(got)


def test_all_six_encodings_and_the_largest_candidate_table():
    x = _tensor("heavy", 20000, 4)
    got, best, want = _run(x, FP8 + FP4, O.FP8_ENCODINGS + O.FP4_ENCODINGS, 170)     # 6 x 170 = 1020 candidates
    np.testing.assert_allclose(got, want, rtol=RTOL, atol=0)
    assert tuple(best) == O.select_encoding_and_bias(got)


def test_full_size_tensor_sampled_candidates():
    # a tensor of the size the bench times (2^24 elements); the oracle checks 2 x 5 of the candidates
    n = 1 << 24
    x = _tensor("normal", n, 5)
    maxabs = float(np.abs(x).max())
    clips = fpq.fpq_search_clip_candidates(maxabs, 111)
    mse, best = fpq.fpq_search_format(torch.from_numpy(x).cuda(), FP8, clips.cuda())
    got = mse.cpu().numpy()
    pick = [0, 27, 55, 99, 110]
    want = O.search_mse(x, [O.FP8_ENCODINGS[1], O.FP8_ENCODINGS[2]], clips.numpy()[pick])
    np.testing.assert_allclose(got[1:3][:, pick], want, rtol=RTOL, atol=0)
    assert tuple(best.cpu().numpy()) == O.select_encoding_and_bias(got)


def test_data_on_a_grid_is_found_with_zero_error():
    f = O.Format(2, 1, 2, O.SAT_PAPER)
    grid = np.array([0, .25, .5, .75, 1, 1.5, 2, 3])
    rng = np.random.default_rng(8)
    x = (rng.choice(grid, 5000) * rng.choice([-1, 1], 5000) * 0.5).astype(np.float32)
    x[0] = 1.5
    got, best, want = _run(x, FP4, O.FP4_ENCODINGS, 6)
    assert got[1, 5] == 0.0 and tuple(best) == (1, 5)
    np.testing.assert_allclose(got, want, rtol=RTOL, atol=0)


def test_empty_tensor_and_nan_and_rejections():
    clips = torch.tensor([1.0, 2.0], device="cuda")
    mse, best = fpq.fpq_search_format(torch.empty(0, device="cuda"), FP4, clips)
    assert (mse.cpu().numpy() == 0).all() and tuple(best.cpu().numpy()) == (0, 0)
    x = torch.tensor([1.0, float("nan"), 2.0], device="cuda")
    mse, best = fpq.fpq_search_format(x, FP4, clips)
    assert fpq.fpq_read_status() == fpq.ERR_NAN_INPUT
    assert np.isnan(mse.cpu().numpy()).all() and tuple(best.cpu().numpy()) == (-1, -1)
    with pytest.raises(Exception):
        fpq.fpq_search_format(x, [fpq.E4M3], clips)            # native saturation is not searched
    with pytest.raises(Exception):
        fpq.fpq_search_format(x, FP8, torch.ones(257, device="cuda"))
    assert fpq.fpq_search_workspace_size(9, 4) == 0 and fpq.fpq_search_workspace_size(8, 129) == 0
