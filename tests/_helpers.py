"""Shared plumbing of the GPU parity tests: run a layer through the C-ABI binding and
through the CPU oracle on the same seeded tensors."""
import numpy as np
import torch

import oracle as O
import paper_2408_06995_b200 as fpq
from paper_2408_06995_b200 import build as fpq_build

fpq_build.build()

FMT = {"e4m3": (fpq.E4M3, O.E4M3), "e2m1": (fpq.E2M1, O.E2M1), "e5m2": (fpq.E5M2, O.E5M2),
       # weight formats that the layer re-encodes exactly into E4M3 when the weights are prepared
       "e1m2": (fpq.E1M2, O.E1M2),
       "e2m1b2": (fpq.Format(2, 1, 2, fpq.SAT_PAPER), O.Format(2, 1, 2, O.SAT_PAPER)),
       "e3m2b3": (fpq.Format(3, 2, 3, fpq.SAT_PAPER), O.Format(3, 2, 3, O.SAT_PAPER)),
       "e2m3b1": (fpq.Format(2, 3, 1, fpq.SAT_PAPER), O.Format(2, 3, 1, O.SAT_PAPER))}


def to_oracle(f: fpq.Format) -> O.Format:
    return O.Format(f.exp_bits, f.man_bits, f.exp_bias, f.sat_mode)


def layer_scales(L):
    """max-scaling per output channel / per tensor; each side divides with its own routine."""
    gfw, ofw = FMT[L.wfmt]
    w2 = L.w.reshape(L.N, -1)
    wmax = np.abs(w2).max(axis=1)
    xmax = float(np.abs(L.x).max())
    ws_o = np.array([O.scale_from_max(v, ofw) for v in wmax], dtype=np.float32)
    xs_o = O.scale_from_max(xmax, O.E4M3)
    ws_g = np.array([fpq.fpq_scale_from_max(float(v), gfw) for v in wmax], dtype=np.float32)
    xs_g = fpq.fpq_scale_from_max(xmax, fpq.E4M3)
    assert np.array_equal(ws_o, ws_g) and np.float32(xs_o) == np.float32(xs_g)
    return ws_g, xs_g


def gpu_prepare(L, ws):
    """Weight encode + contraction-ready copy on the GPU; returns (codes, prepared)."""
    gfw, _ = FMT[L.wfmt]
    dev = "cuda"
    w2 = torch.from_numpy(L.w.reshape(L.N, -1)).to(dev)
    rb = None
    if L.bits is not None:
        rb = torch.from_numpy(O.pack_bits(L.bits)).to(dev)
    codes = fpq.fpq_quantize_weight(w2, torch.from_numpy(ws).to(dev), gfw, rb)
    if L.kind == "linear":
        prep = fpq.fpq_prepare_weight(codes, gfw, fpq.LINEAR, L.N, L.K)
    else:
        prep = fpq.fpq_prepare_weight(codes, gfw, fpq.CONV2D, L.N, L.C, L.R, L.S)
    return codes, prep


GUARD = 256          # bytes of guard band on each side of an output or workspace buffer
CANARY = 0xA5        # every guard byte (as FP32 words: 0xA5A5A5A5, a pattern no result produces)


class Guarded:
    """A device buffer with a guard band in front of it and behind it.  The library gets the inner view; after
    the call the bands must still hold the canary bytes: a store one element before or past a ragged output,
    or past the workspace size the library itself asked for, is caught on the host."""

    def __init__(self, nbytes, dev="cuda"):
        self.n = int(nbytes)
        pad = (-self.n) % 256                          # the band behind starts on a 256-byte boundary
        self.raw = torch.full((GUARD + self.n + pad + GUARD,), CANARY, dtype=torch.uint8, device=dev)
        self.inner = self.raw[GUARD:GUARD + self.n]

    def f32(self, shape):
        return self.inner.view(torch.float32).view(shape)

    def check(self, what):
        front = self.raw[:GUARD]
        back = self.raw[GUARD + self.n:]
        assert bool((front == CANARY).all()), f"{what}: bytes in front of the buffer were overwritten"
        assert bool((back == CANARY).all()), f"{what}: bytes behind the buffer were overwritten"


def _gpu_layer_once(L, ws, xs, use_bias, prep):
    gfw, _ = FMT[L.wfmt]
    dev = "cuda"
    x = torch.from_numpy(L.x).to(dev)
    bias = torch.from_numpy(L.bias).to(dev) if use_bias else None
    wsd = torch.from_numpy(ws).to(dev)
    if L.kind == "linear":
        yg = Guarded(4 * L.M * L.N)
        wg = Guarded(max(1, fpq.fpq_linear_workspace_size(L.M, L.N, L.K, fpq.E4M3, gfw)))
        y = fpq.fpq_linear(x, prep, wsd, xs, fpq.E4M3, gfw, bias, L.N, y=yg.f32((L.M, L.N)), workspace=wg.inner)
    else:
        yg = Guarded(4 * L.B * L.N * L.Ho * L.Wo)
        wg = Guarded(max(1, fpq.fpq_conv2d_workspace_size(L.B, L.C, L.H, L.W, L.N, L.R, L.S, L.pad, L.stride,
                                                           fpq.E4M3, gfw)))
        y = fpq.fpq_conv2d(x, prep, wsd, xs, fpq.E4M3, gfw, bias, L.N, L.R, L.S, L.pad, L.stride,
                           y=yg.f32((L.B, L.N, L.Ho, L.Wo)), workspace=wg.inner)
    st = fpq.fpq_read_status()
    assert st == fpq.OK, fpq.status_string(st)
    yg.check(f"{L.name} output")
    wg.check(f"{L.name} workspace")
    return y.cpu().numpy()


def gpu_layer(L, ws, xs, use_bias=True, route="auto"):
    """The layer call on every route of the library (one fused kernel; quantize kernel + contraction kernel;
    the library's own choice).  All routes multiply the same codes exactly and add in FP32; where they run the
    same MMAs in the same order the results are equal bit for bit, otherwise (a fused kernel that splits the
    reduction differently) they differ by the rounding of the FP32 sums only.  The library's own choice must be
    one of the two, bit for bit.  Returns the result of `route` ("auto", "fused" or "two")."""
    _, prep = gpu_prepare(L, ws)
    try:
        fpq.fpq_set_path_policy(fpq.PATH_FUSED)
        y1 = _gpu_layer_once(L, ws, xs, use_bias, prep)
        fpq.fpq_set_path_policy(fpq.PATH_TWO_KERNELS)
        y2 = _gpu_layer_once(L, ws, xs, use_bias, prep)
    finally:
        fpq.fpq_set_path_policy(fpq.PATH_AUTO)
    y0 = _gpu_layer_once(L, ws, xs, use_bias, prep)
    assert np.array_equal(y0, y1) or np.array_equal(y0, y2), "the default route is neither of the two routes"
    if not np.array_equal(y1, y2):
        scale = float(np.abs(y2).max()) if y2.size else 0.0
        assert np.all(np.abs(y1.astype(np.float64) - y2) <= 1e-4 * scale), "fused and two-kernel routes differ"
    return {"auto": y0, "fused": y1, "two": y2}[route]


def oracle_layer(L, ws, xs, idx=None, use_bias=True):
    _, ofw = FMT[L.wfmt]
    rb = O.pack_bits(L.bits) if L.bits is not None else None
    bias = L.bias if use_bias else None
    if L.kind == "linear":
        return O.linear(L.x, L.w, ws, xs, O.E4M3, ofw, bias, rb, idx)
    return O.conv2d(L.x, L.w, ws, xs, O.E4M3, ofw, bias, rb, L.pad, L.stride, idx)


def assert_close(y_gpu, y_ref, absum):
    """|err| <= 1e-3 * sum_k |a_k b_k| per output element, plus two FP32 ulps of |y|
    for the final scale-and-bias rounding."""
    y_gpu = np.asarray(y_gpu, dtype=np.float64).reshape(-1)
    y_ref = np.asarray(y_ref).reshape(-1)
    absum = np.asarray(absum).reshape(-1)
    tol = 1e-3 * absum + 2.0 * np.spacing(np.abs(y_ref).astype(np.float32)).astype(np.float64)
    err = np.abs(y_gpu - y_ref)
    worst = int(np.argmax(err - tol))
    assert np.all(err <= tol), (worst, y_gpu[worst], y_ref[worst], err[worst], tol[worst])
    return float((err / np.maximum(absum, 1e-30)).max())


def sample_indices(total, n, seed, extra=()):
    rng = np.random.default_rng(seed)
    idx = rng.integers(0, total, size=n, dtype=np.int64)
    idx = np.unique(np.concatenate([idx, np.asarray(extra, dtype=np.int64)]))
    return idx
