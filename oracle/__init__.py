"""CPU oracle (test infrastructure only).

Thin numpy/ctypes front end of ``fpq_oracle.c``: the plain definition of the
paper's floating-point quantizer (Sec. IV-B), its learned-rounding variant with
hardened decisions (Sec. V-B), the quantized linear / conv layer (Sec. V-B,
Sec. VI-A), summed in double, the encoding / bias search (Sec. V-A) and one
evaluation of the rounding-learning objective and its gradient (Sec. V-B).  Nothing in the product path may import this
package: it exists so that tests, the smoke check and the benchmark's
CPU-baseline leg have something independent to compare the CUDA library with.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fpq_oracle.c")
_SO = os.path.join(_HERE, "libfpq_oracle.so")

SAT_PAPER = 0
SAT_NATIVE = 1


@dataclass(frozen=True)
class Format:
    """(exponent bits, mantissa bits, integer exponent bias, saturation mode)."""

    e: int
    m: int
    B: int
    sat: int = SAT_PAPER

    @property
    def bits(self) -> int:
        return 4 if 1 + self.e + self.m <= 4 else 8


E4M3 = Format(4, 3, 7, SAT_NATIVE)
E5M2 = Format(5, 2, 15, SAT_NATIVE)
E2M1 = Format(2, 1, 1, SAT_PAPER)
E1M2 = Format(1, 2, 1, SAT_PAPER)
E3M4 = Format(3, 4, 4, SAT_PAPER)
E2M5 = Format(2, 5, 2, SAT_PAPER)


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C, OpenMP over output rows)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fno-fast-math", "-fPIC",
               "-shared", _SRC, "-o", _SO, "-lm"]
        subprocess.run(cmd, check=True)
    return _SO


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        i32, i64, f32, f64 = ctypes.c_int32, ctypes.c_int64, ctypes.c_float, ctypes.c_double
        vp = ctypes.c_void_p
        L.fpq_o_decode.restype = f64
        L.fpq_o_decode.argtypes = [i32, i32, i32, i32]
        L.fpq_o_cmax.restype = f64
        L.fpq_o_cmax.argtypes = [i32, i32, i32, i32]
        L.fpq_o_quantize_one.restype = i32
        L.fpq_o_quantize_one.argtypes = [f32, f32, i32, i32, i32, i32, i32, vp]
        L.fpq_o_quantize_weight.restype = i64
        L.fpq_o_quantize_weight.argtypes = [vp, i64, i64, vp, i32, i32, i32, i32, vp, vp]
        L.fpq_o_quantize_act.restype = i64
        L.fpq_o_quantize_act.argtypes = [vp, i64, f32, i32, i32, i32, i32, vp]
        L.fpq_o_linear.restype = i32
        L.fpq_o_linear.argtypes = [vp, vp, vp, f32, i32, i32, i32, i32, i32, i32, vp, i64, i64, i64,
                                   vp, i64, vp, vp]
        L.fpq_o_conv2d.restype = i32
        L.fpq_o_conv2d.argtypes = [vp, vp, vp, f32, i32, i32, i32, i32, i32, i32, vp,
                                   i64, i64, i64, i64, i64, i64, i64, i64, i64, vp, i64, vp, vp]
        L.fpq_o_search_mse.restype = i64
        L.fpq_o_search_mse.argtypes = [vp, i64, vp, i32, vp, i32, vp]
        L.fpq_o_soft_weight.restype = i64
        L.fpq_o_soft_weight.argtypes = [vp, i64, i64, vp, i32, i32, i32, i32, vp, vp, vp]
        _lib = L
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def decode(code: int, f: Format) -> float:
    return lib().fpq_o_decode(int(code), f.e, f.m, f.B)


def decode_table(f: Format) -> np.ndarray:
    """Values of all 2^(1+e+m) codes, indexed by code."""
    return np.array([decode(c, f) for c in range(1 << (1 + f.e + f.m))], dtype=np.float64)


def cmax(f: Format) -> float:
    return lib().fpq_o_cmax(f.e, f.m, f.B, f.sat)


def scale_from_max(maxabs: float, f: Format) -> np.float32:
    """Scale that maps maxabs onto the clipping value: FP32 division."""
    return np.float32(np.float32(maxabs) / np.float32(cmax(f)))


def quantize_one(x: float, scale: float, f: Format, h: int = -1) -> int:
    return lib().fpq_o_quantize_one(float(np.float32(x)), float(np.float32(scale)), f.e, f.m, f.B,
                                    f.sat, int(h), None)


def pack_bits(bits01: np.ndarray) -> np.ndarray:
    """[N][K] array of 0/1 -> [N][ceil(K/8)] bytes, LSB first along K."""
    return np.packbits(np.ascontiguousarray(bits01, dtype=np.uint8), axis=1, bitorder="little")


def quantize_weight(w, scale, f: Format, rounding_bits=None) -> np.ndarray:
    """w: [N][K] (conv weights flattened to [Co][C*R*S]); scale: [N];
    rounding_bits: packed bytes from pack_bits or None for round to nearest."""
    w = _f32(w)
    N, K = w.shape
    scale = _f32(scale)
    assert scale.shape == (N,)
    row = K if f.bits == 8 else (K + 1) // 2
    codes = np.zeros((N, row), dtype=np.uint8)
    rb = None
    if rounding_bits is not None:
        rb = np.ascontiguousarray(rounding_bits, dtype=np.uint8)
        assert rb.shape == (N, (K + 7) // 8)
    lib().fpq_o_quantize_weight(_p(w), N, K, _p(scale), f.e, f.m, f.B, f.sat, _p(rb), _p(codes))
    return codes


def quantize_act(x, scale, f: Format) -> np.ndarray:
    x = _f32(x)
    n = x.size
    codes = np.zeros(n if f.bits == 8 else (n + 1) // 2, dtype=np.uint8)
    lib().fpq_o_quantize_act(_p(x), n, float(np.float32(scale)), f.e, f.m, f.B, f.sat, _p(codes))
    return codes.reshape(x.shape) if f.bits == 8 else codes


def linear_codes(xc, wc, w_scale, x_scale, fx: Format, fw: Format, bias, M, N, K, idx=None):
    """Returns (y, absum) in double; with idx only those flat positions i*N+n."""
    xc = np.ascontiguousarray(xc, dtype=np.uint8)
    wc = np.ascontiguousarray(wc, dtype=np.uint8)
    w_scale = _f32(w_scale)
    bias = None if bias is None else _f32(bias)
    if idx is not None:
        idx = np.ascontiguousarray(idx, dtype=np.int64)
        n_out = idx.size
    else:
        n_out = M * N
    y = np.zeros(n_out, dtype=np.float64)
    ab = np.zeros(n_out, dtype=np.float64)
    rc = lib().fpq_o_linear(_p(xc), _p(wc), _p(w_scale), float(np.float32(x_scale)), fx.e, fx.m,
                            fx.B, fw.e, fw.m, fw.B, _p(bias), M, N, K, _p(idx),
                            0 if idx is None else idx.size, _p(y), _p(ab))
    assert rc == 0
    if idx is None:
        return y.reshape(M, N), ab.reshape(M, N)
    return y, ab


def conv2d_codes(xc, wc, w_scale, x_scale, fx: Format, fw: Format, bias, B, C, H, W, Co, R, S, pad,
                 stride, idx=None):
    xc = np.ascontiguousarray(xc, dtype=np.uint8)
    wc = np.ascontiguousarray(wc, dtype=np.uint8)
    w_scale = _f32(w_scale)
    bias = None if bias is None else _f32(bias)
    Ho = (H + 2 * pad - R) // stride + 1
    Wo = (W + 2 * pad - S) // stride + 1
    if idx is not None:
        idx = np.ascontiguousarray(idx, dtype=np.int64)
        n_out = idx.size
    else:
        n_out = B * Co * Ho * Wo
    y = np.zeros(n_out, dtype=np.float64)
    ab = np.zeros(n_out, dtype=np.float64)
    rc = lib().fpq_o_conv2d(_p(xc), _p(wc), _p(w_scale), float(np.float32(x_scale)), fx.e, fx.m,
                            fx.B, fw.e, fw.m, fw.B, _p(bias), B, C, H, W, Co, R, S, pad, stride,
                            _p(idx), 0 if idx is None else idx.size, _p(y), _p(ab))
    assert rc == 0
    if idx is None:
        return y.reshape(B, Co, Ho, Wo), ab.reshape(B, Co, Ho, Wo)
    return y, ab


def linear(x, w, w_scale, x_scale, fx: Format, fw: Format, bias=None, rounding_bits=None, idx=None):
    """The whole quantized linear layer from FP32 inputs: quantize weights
    (first) and activations (Sec. VI-A), contract, rescale, add bias."""
    x = _f32(x)
    w = _f32(w)
    M, K = x.shape
    N = w.shape[0]
    wc = quantize_weight(w, w_scale, fw, rounding_bits)
    xc = quantize_act(x, x_scale, fx)
    return linear_codes(xc, wc, w_scale, x_scale, fx, fw, bias, M, N, K, idx)


def conv2d(x, w, w_scale, x_scale, fx: Format, fw: Format, bias=None, rounding_bits=None, pad=0,
           stride=1, idx=None):
    """The whole quantized conv layer from FP32 NCHW input and [Co][C][R][S] weights."""
    x = _f32(x)
    w = _f32(w)
    B, C, H, W = x.shape
    Co, C2, R, S = w.shape
    assert C2 == C
    wc = quantize_weight(w.reshape(Co, C * R * S), w_scale, fw, rounding_bits)
    xc = quantize_act(x, x_scale, fx)
    return conv2d_codes(xc, wc, w_scale, x_scale, fx, fw, bias, B, C, H, W, Co, R, S, pad, stride, idx)


# ---- encoding and bias search (Sec. V-A, Algorithm 1) -------------------------------------

FP8_ENCODINGS = (E2M5, E3M4, Format(4, 3, 8, SAT_PAPER), Format(5, 2, 16, SAT_PAPER))   # bias 2^(e-1), Sec. IV-B
FP4_ENCODINGS = (E1M2, Format(2, 1, 2, SAT_PAPER))


def clip_candidates(maxabs: float, count: int = 111) -> np.ndarray:
    """Evenly spaced clipping values up to the largest magnitude of the data (Sec. V-A):
    c_j = maxabs * j / count for j = 1..count, rounded once to FP32.  (Zero is left out: no
    format has c = 0.)"""
    return np.array([np.float32(float(np.float32(maxabs)) * j / count) for j in range(1, count + 1)],
                    dtype=np.float32)


def bias_from_clip(c: float, f: Format) -> float:
    """The real-valued exponent bias whose clipping value is c: the clipping equation
    c = (2 - 2^-m) 2^(2^e - b - 1) solved for b (Sec. IV-B)."""
    return float(2 ** f.e - 1 - np.log2(float(c) / (2.0 - 2.0 ** -f.m)))


def search_mse(x, encodings, clips) -> np.ndarray:
    """mse[i][j] of quantizing x with encoding i clipped at clips[j] (see fpq_o_search_mse)."""
    x = _f32(x).reshape(-1)
    enc = np.ascontiguousarray([[f.e, f.m, f.B] for f in encodings], dtype=np.int32)
    clips = _f32(clips)
    mse = np.zeros((len(encodings), clips.size), dtype=np.float64)
    lib().fpq_o_search_mse(_p(x), x.size, _p(enc), len(encodings), _p(clips), clips.size, _p(mse))
    return mse


def select_encoding_and_bias(mse: np.ndarray):
    """The selection rule of Algorithm 1 (Sec. V-A): the (encoding, bias candidate) pair with the smallest
    error; among equal errors the first one in encoding-major, candidate-minor order.  The listing prints a
    start value of 0 for the best error so far, which no candidate could ever beat: read as +infinity.  A
    NaN error is never selected, and with no finite-or-infinite error below +infinity nothing is selected."""
    m = np.asarray(mse, dtype=np.float64)
    flat = np.where(np.isnan(m), np.inf, m).reshape(-1)
    if flat.size == 0 or not np.any(flat < np.inf):
        return (None, None)
    k = int(np.argmin(flat))                      # argmin returns the first occurrence of the minimum
    return (k // m.shape[1], k % m.shape[1])


# ---- sparsity of a quantized tensor (the paper's sparsity study) --------------------------

def zero_count(codes, n: int, f: Format) -> int:
    """How many of the n quantized values are zero (code 0: the quantizer has no negative zero).
    `codes` is laid out as quantize_weight / quantize_act write it."""
    flat = np.ascontiguousarray(codes, dtype=np.uint8).reshape(-1)
    if f.bits == 8:
        return int(np.count_nonzero(flat[:n] == 0))
    values = np.empty(flat.size * 2, dtype=np.uint8)
    values[0::2] = flat & 0xF
    values[1::2] = flat >> 4
    return int(np.count_nonzero(values[:n] == 0))


# ---- rounding learning (Sec. V-B) -----------------------------------------------------------


def soft_weight(w, scale, f: Format, alpha):
    """Soft-rounded weights W^q(alpha) of the learned-rounding equation (Sec. V-B) and their
    derivative with respect to alpha, both [N][K] float64."""
    w = _f32(w)
    alpha = _f32(alpha)
    scale = _f32(scale)
    N, K = w.shape
    assert alpha.shape == (N, K) and scale.shape == (N,)
    wq = np.zeros((N, K), dtype=np.float64)
    dwq = np.zeros((N, K), dtype=np.float64)
    lib().fpq_o_soft_weight(_p(w), N, K, _p(scale), f.e, f.m, f.B, f.sat, _p(alpha), _p(wq), _p(dwq))
    return wq, dwq


def rounding_regularizer(alpha):
    """lambda(alpha) = 1 - (2 |sigma(alpha) - 0.5|)^20 per element (Sec. V-B) and its derivative."""
    al = np.asarray(alpha, dtype=np.float64)
    sig = 1.0 / (1.0 + np.exp(-al))
    u = 2.0 * np.abs(sig - 0.5)
    lam = 1.0 - u ** 20
    dlam = -20.0 * u ** 19 * 2.0 * np.sign(sig - 0.5) * sig * (1.0 - sig)
    return lam, dlam


def round_learn_loss(w, scale, f: Format, alpha, a, reg: float):
    """The rounding-learning objective of Sec. V-B for a bias-free linear layer with calibration
    activations a [M][K]:  mean((A W^q(alpha)^T - A W^T)^2) + reg * sum_i lambda(alpha_i).
    Returns (mse, sum of lambda)."""
    w64 = np.asarray(_f32(w), dtype=np.float64)
    a64 = np.asarray(_f32(a), dtype=np.float64)
    wq, _ = soft_weight(w, scale, f, alpha)
    y = a64 @ w64.T
    yq = a64 @ wq.T
    lam, _ = rounding_regularizer(_f32(alpha))
    return float(np.mean((yq - y) ** 2)), float(lam.sum())


def round_learn_step(w, scale, f: Format, alpha, a, reg: float):
    """One evaluation of the objective and of its gradient with respect to alpha.
    Chain rule on the definition: d mse / d W^q = (2 / (M N)) (Y^q - Y)^T A, times the element's
    own d W^q / d alpha, plus reg * d lambda / d alpha.  Also returns the per-element sum of
    absolute terms of the gradient's contraction (for the parity tolerance)."""
    w64 = np.asarray(_f32(w), dtype=np.float64)
    a64 = np.asarray(_f32(a), dtype=np.float64)
    M = a64.shape[0]
    N = w64.shape[0]
    wq, dwq = soft_weight(w, scale, f, alpha)
    y = a64 @ w64.T
    yq = a64 @ wq.T
    d = yq - y
    mse = float(np.mean(d ** 2))
    lam, dlam = rounding_regularizer(_f32(alpha))
    g = (2.0 / (M * N)) * (d.T @ a64)
    grad = g * dwq + reg * dlam
    absum = (2.0 / (M * N)) * (np.abs(d).T @ np.abs(a64)) * np.abs(dwq)
    return {"mse": mse, "reg": float(lam.sum()), "grad": grad, "absum": absum, "wq": wq, "d": d}


def unfold(x, R: int, S: int, pad: int, stride: int) -> np.ndarray:
    """Input rows of a convolution (Sec. V-B applies the learning step to convolutions as well): row
    (b, oy, ox), column (c, r, s) = x[b][c][oy*stride - pad + r][ox*stride - pad + s], zero in the padding.
    Plain loops over the window."""
    x = _f32(x)
    B, C, H, W = x.shape
    Ho, Wo = (H + 2 * pad - R) // stride + 1, (W + 2 * pad - S) // stride + 1
    xp = np.zeros((B, C, H + 2 * pad, W + 2 * pad), dtype=np.float32)
    xp[:, :, pad:pad + H, pad:pad + W] = x
    rows = np.zeros((B, Ho, Wo, C, R, S), dtype=np.float32)
    for oy in range(Ho):
        for ox in range(Wo):
            for r in range(R):
                for s in range(S):
                    rows[:, oy, ox, :, r, s] = xp[:, :, oy * stride + r, ox * stride + s]
    return rows.reshape(B * Ho * Wo, C * R * S)
