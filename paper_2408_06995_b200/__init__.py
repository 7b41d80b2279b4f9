"""Python binding of libfpq.so: argument marshalling only.

Every function here has the name of the C entry point it calls
(include/fpq.h) and passes torch tensors' device pointers and the current CUDA
stream.  All arithmetic runs in the library's kernels.  There is no fallback:
if the shared library is missing the import of a symbol fails.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "libfpq.so")

OK = 0
ERR_NULL, ERR_FORMAT, ERR_SHAPE, ERR_ALIGN, ERR_UNSUPPORTED = -1, -2, -3, -4, -5
ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT, ERR_NAN_INPUT, ERR_TOO_LARGE, ERR_SCALE = -6, -7, -8, -9, -10, -11
ROUTE_TWO_KERNELS, ROUTE_FUSED, ROUTE_PAIR_FUSED, ROUTE_OTHER = 0, 1, 2, 3
STATIC_SCRATCH_BYTES = 8 << 20
SAT_PAPER, SAT_NATIVE = 0, 1
LINEAR, CONV2D = 0, 1
PATH_AUTO, PATH_FUSED, PATH_TWO_KERNELS, PATH_TWO_KERNELS_NARROW = 0, 1, 2, 3


class FpqError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} ({code})")


class _CFormat(ctypes.Structure):
    _fields_ = [("exp_bits", ctypes.c_int32), ("man_bits", ctypes.c_int32),
                ("exp_bias", ctypes.c_int32), ("sat_mode", ctypes.c_int32)]


class _CLayerDesc(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int32), ("N", ctypes.c_int32), ("C", ctypes.c_int32),
                ("R", ctypes.c_int32), ("S", ctypes.c_int32)]


@dataclass(frozen=True)
class Format:
    exp_bits: int
    man_bits: int
    exp_bias: int
    sat_mode: int = SAT_PAPER

    def c(self) -> _CFormat:
        return _CFormat(self.exp_bits, self.man_bits, self.exp_bias, self.sat_mode)

    @property
    def four_bit(self) -> bool:
        return 1 + self.exp_bits + self.man_bits <= 4


E4M3 = Format(4, 3, 7, SAT_NATIVE)
E5M2 = Format(5, 2, 15, SAT_NATIVE)
E2M1 = Format(2, 1, 1, SAT_PAPER)
E1M2 = Format(1, 2, 1, SAT_PAPER)
E3M4 = Format(3, 4, 4, SAT_PAPER)
E2M5 = Format(2, 5, 2, SAT_PAPER)

EXPORTS = [
    "fpq_scale_from_max", "fpq_format_max", "fpq_quantize_weight", "fpq_quantize_act",
    "fpq_prepared_size", "fpq_prepare_weight", "fpq_linear_workspace_size", "fpq_linear",
    "fpq_conv2d_workspace_size", "fpq_conv2d", "fpq_linear_host", "fpq_conv2d_host",
    "fpq_linear_quantize_input", "fpq_linear_contract", "fpq_conv2d_quantize_input", "fpq_conv2d_contract",
    "fpq_linear_static", "fpq_search_workspace_size", "fpq_search_format", "fpq_search_clip_candidates",
    "fpq_round_learn_workspace_size", "fpq_round_learn_step", "fpq_round_learn_harden", "fpq_round_learn_unfold",
    "fpq_zero_census", "fpq_prepared_size_split", "fpq_prepare_weight_split", "fpq_conv2d_split_workspace_size",
    "fpq_conv2d_split", "fpq_set_path_policy", "fpq_get_path_policy", "fpq_read_status", "fpq_status_string",
    "fpq_conv2d_route", "fpq_selftest_bounded_wait",
]

_lib = None


def lib() -> ctypes.CDLL:
    """The loaded shared library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(_SO):
            raise FileNotFoundError(
                f"{_SO} is missing: build it with `python -m paper_2408_06995_b200.build` "
                "(there is no CPU or PyTorch fallback)")
        L = ctypes.CDLL(_SO)
        i32, i64, f32 = ctypes.c_int32, ctypes.c_int64, ctypes.c_float
        vp, sz = ctypes.c_void_p, ctypes.c_size_t
        F, D = _CFormat, ctypes.POINTER(_CLayerDesc)
        L.fpq_round_learn_workspace_size.restype = sz
        L.fpq_round_learn_workspace_size.argtypes = [i64, i64, i64]
        L.fpq_round_learn_step.restype = i32
        L.fpq_round_learn_step.argtypes = [vp, vp, F, vp, vp, i64, i64, i64, f32, f32, vp, vp, vp, sz, vp]
        L.fpq_round_learn_unfold.restype = i32
        L.fpq_round_learn_unfold.argtypes = [vp, i32, i32, i32, i32, i32, i32, i32, i32, vp, vp]
        L.fpq_round_learn_harden.restype = i32
        L.fpq_round_learn_harden.argtypes = [vp, i64, i64, vp, vp]
        L.fpq_scale_from_max.restype = f32
        L.fpq_scale_from_max.argtypes = [f32, F]
        L.fpq_format_max.restype = f32
        L.fpq_format_max.argtypes = [F]
        L.fpq_quantize_weight.restype = i32
        L.fpq_quantize_weight.argtypes = [vp, i64, i64, vp, F, vp, vp, vp]
        L.fpq_quantize_act.restype = i32
        L.fpq_quantize_act.argtypes = [vp, i64, f32, F, vp, vp]
        L.fpq_prepared_size.restype = sz
        L.fpq_prepared_size.argtypes = [F, D]
        L.fpq_prepare_weight.restype = i32
        L.fpq_prepare_weight.argtypes = [vp, F, D, vp, vp]
        L.fpq_linear_workspace_size.restype = sz
        L.fpq_linear_workspace_size.argtypes = [i64, i64, i64, F, F]
        L.fpq_linear.restype = i32
        L.fpq_linear.argtypes = [vp, vp, vp, f32, F, F, vp, vp, i64, i64, i64, vp, sz, vp]
        L.fpq_conv2d_workspace_size.restype = sz
        L.fpq_conv2d_workspace_size.argtypes = [i32] * 9 + [F, F]
        L.fpq_conv2d.restype = i32
        L.fpq_conv2d.argtypes = [vp, vp, vp, f32, F, F, vp, vp] + [i32] * 9 + [vp, sz, vp]
        L.fpq_linear_host.restype = i32
        L.fpq_linear_host.argtypes = [vp, vp, vp, vp, f32, F, F, vp, vp, vp, i64, i64, i64, vp, sz, vp]
        L.fpq_conv2d_host.restype = i32
        L.fpq_conv2d_host.argtypes = [vp, vp, vp, vp, f32, F, F, vp, vp, vp] + [i32] * 9 + [vp, sz, vp]
        L.fpq_linear_quantize_input.restype = i32
        L.fpq_linear_quantize_input.argtypes = [vp, f32, F, F, i64, i64, i64, vp, sz, vp]
        L.fpq_linear_contract.restype = i32
        L.fpq_linear_contract.argtypes = [vp, sz, vp, vp, f32, F, F, vp, vp, i64, i64, i64, vp]
        L.fpq_conv2d_quantize_input.restype = i32
        L.fpq_conv2d_quantize_input.argtypes = [vp, f32, F, F] + [i32] * 9 + [vp, sz, vp]
        L.fpq_conv2d_contract.restype = i32
        L.fpq_conv2d_contract.argtypes = [vp, sz, vp, vp, f32, F, F, vp, vp] + [i32] * 9 + [vp]
        L.fpq_linear_static.restype = i32
        L.fpq_linear_static.argtypes = [vp, vp, vp, f32, F, F, vp, vp, i64, i64, i64, vp]
        L.fpq_prepared_size_split.restype = sz
        L.fpq_prepared_size_split.argtypes = [F, i32, i32, i32, i32, i32]
        L.fpq_prepare_weight_split.restype = i32
        L.fpq_prepare_weight_split.argtypes = [vp, F, i32, i32, i32, i32, i32, vp, vp]
        L.fpq_conv2d_split_workspace_size.restype = sz
        L.fpq_conv2d_split_workspace_size.argtypes = [i32] * 10 + [F, F]
        L.fpq_conv2d_split.restype = i32
        L.fpq_conv2d_split.argtypes = [vp, i32, f32, vp, i32, f32, vp, vp, F, F, vp, vp] + [i32] * 8 + [vp, sz, vp]
        L.fpq_zero_census.restype = i32
        L.fpq_zero_census.argtypes = [vp, i64, F, vp, vp]
        L.fpq_search_workspace_size.restype = sz
        L.fpq_search_workspace_size.argtypes = [i32, i32]
        L.fpq_search_format.restype = i32
        L.fpq_search_format.argtypes = [vp, i64, vp, i32, vp, i32, vp, vp, vp, sz, vp]
        L.fpq_search_clip_candidates.restype = i32
        L.fpq_search_clip_candidates.argtypes = [f32, i32, vp]
        L.fpq_set_path_policy.restype = i32
        L.fpq_set_path_policy.argtypes = [i32]
        L.fpq_get_path_policy.restype = i32
        L.fpq_get_path_policy.argtypes = []
        L.fpq_selftest_bounded_wait.restype = i32
        L.fpq_selftest_bounded_wait.argtypes = [i64, vp]
        L.fpq_conv2d_route.restype = i32
        L.fpq_conv2d_route.argtypes = [i32] * 9 + [F, F]
        L.fpq_read_status.restype = i32
        L.fpq_read_status.argtypes = [vp]
        L.fpq_status_string.restype = ctypes.c_char_p
        L.fpq_status_string.argtypes = [i32]
        _lib = L
    return _lib


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(code: int, where: str):
    if code != OK:
        raise FpqError(code, where)


def status_string(code: int) -> str:
    return lib().fpq_status_string(int(code)).decode()


def fpq_format_max(fmt: Format) -> float:
    return lib().fpq_format_max(fmt.c())


def fpq_scale_from_max(maxabs: float, fmt: Format) -> float:
    return lib().fpq_scale_from_max(float(maxabs), fmt.c())


def fpq_quantize_weight(w: torch.Tensor, scale: torch.Tensor, fmt: Format, rounding_bits=None,
                        codes: torch.Tensor = None) -> torch.Tensor:
    """w [N][K] float32 (cuda, contiguous), scale [N], rounding_bits packed uint8
    [N][ceil(K/8)] or None.  Returns codes [N][K] or [N][ceil(K/2)] uint8."""
    assert w.is_cuda and w.dtype == torch.float32 and w.is_contiguous() and w.dim() == 2
    N, K = w.shape
    if codes is None:
        codes = torch.empty((N, (K + 1) // 2 if fmt.four_bit else K), dtype=torch.uint8, device=w.device)
    _check(lib().fpq_quantize_weight(_ptr(w), N, K, _ptr(scale), fmt.c(), _ptr(rounding_bits), _ptr(codes),
                                     _stream()), "fpq_quantize_weight")
    return codes


def fpq_quantize_act(x: torch.Tensor, scale: float, fmt: Format, codes: torch.Tensor = None) -> torch.Tensor:
    assert x.is_cuda and x.dtype == torch.float32 and x.is_contiguous()
    n = x.numel()
    if codes is None:
        shape = ((n + 1) // 2,) if fmt.four_bit else tuple(x.shape)
        codes = torch.empty(shape, dtype=torch.uint8, device=x.device)
    _check(lib().fpq_quantize_act(_ptr(x), n, float(scale), fmt.c(), _ptr(codes), _stream()), "fpq_quantize_act")
    return codes


def _desc(kind, N, C, R=1, S=1):
    return _CLayerDesc(kind, N, C, R, S)


def fpq_prepared_size(fmt: Format, kind: int, N: int, C: int, R: int = 1, S: int = 1) -> int:
    d = _desc(kind, N, C, R, S)
    return lib().fpq_prepared_size(fmt.c(), ctypes.byref(d))


def fpq_prepare_weight(codes: torch.Tensor, fmt: Format, kind: int, N: int, C: int, R: int = 1, S: int = 1,
                       prepared: torch.Tensor = None) -> torch.Tensor:
    d = _desc(kind, N, C, R, S)
    size = lib().fpq_prepared_size(fmt.c(), ctypes.byref(d))
    if size == 0:
        raise FpqError(ERR_SHAPE, "fpq_prepared_size")
    if prepared is None:
        prepared = torch.empty(size, dtype=torch.uint8, device=codes.device)
    _check(lib().fpq_prepare_weight(_ptr(codes), fmt.c(), ctypes.byref(d), _ptr(prepared), _stream()),
           "fpq_prepare_weight")
    return prepared


def fpq_linear_workspace_size(M, N, K, fx: Format, fw: Format) -> int:
    return lib().fpq_linear_workspace_size(M, N, K, fx.c(), fw.c())


def fpq_linear(x, w_prepared, w_scale, x_scale, fx: Format, fw: Format, bias, N: int, y=None, workspace=None):
    assert x.is_cuda and x.dtype == torch.float32 and x.is_contiguous() and x.dim() == 2
    M, K = x.shape
    if y is None:
        y = torch.empty((M, N), dtype=torch.float32, device=x.device)
    if workspace is None:
        workspace = torch.empty(max(1, fpq_linear_workspace_size(M, N, K, fx, fw)), dtype=torch.uint8, device=x.device)
    _check(lib().fpq_linear(_ptr(x), _ptr(w_prepared), _ptr(w_scale), float(x_scale), fx.c(), fw.c(), _ptr(bias),
                            _ptr(y), M, N, K, _ptr(workspace), workspace.numel(), _stream()), "fpq_linear")
    return y


def fpq_conv2d_workspace_size(B, C, H, W, C_out, R, S, pad, stride, fx: Format, fw: Format) -> int:
    return lib().fpq_conv2d_workspace_size(B, C, H, W, C_out, R, S, pad, stride, fx.c(), fw.c())


def fpq_conv2d(x, w_prepared, w_scale, x_scale, fx: Format, fw: Format, bias, C_out, R, S, pad, stride, y=None,
               workspace=None):
    assert x.is_cuda and x.dtype == torch.float32 and x.is_contiguous() and x.dim() == 4
    B, C, H, W = x.shape
    Ho = (H + 2 * pad - R) // stride + 1
    Wo = (W + 2 * pad - S) // stride + 1
    if y is None:
        y = torch.empty((B, C_out, Ho, Wo), dtype=torch.float32, device=x.device)
    if workspace is None:
        workspace = torch.empty(max(1, fpq_conv2d_workspace_size(B, C, H, W, C_out, R, S, pad, stride, fx, fw)),
                                dtype=torch.uint8, device=x.device)
    _check(lib().fpq_conv2d(_ptr(x), _ptr(w_prepared), _ptr(w_scale), float(x_scale), fx.c(), fw.c(), _ptr(bias),
                            _ptr(y), B, C, H, W, C_out, R, S, pad, stride, _ptr(workspace), workspace.numel(),
                            _stream()), "fpq_conv2d")
    return y


def fpq_linear_quantize_input(x, x_scale, fx: Format, fw: Format, N: int, workspace):
    M, K = x.shape
    _check(lib().fpq_linear_quantize_input(_ptr(x), float(x_scale), fx.c(), fw.c(), M, N, K, _ptr(workspace),
                                           workspace.numel(), _stream()), "fpq_linear_quantize_input")
    return workspace


def fpq_linear_contract(workspace, w_prepared, w_scale, x_scale, fx: Format, fw: Format, bias, y, K: int):
    M, N = y.shape
    _check(lib().fpq_linear_contract(_ptr(workspace), workspace.numel(), _ptr(w_prepared), _ptr(w_scale),
                                     float(x_scale), fx.c(), fw.c(), _ptr(bias), _ptr(y), M, N, K, _stream()),
           "fpq_linear_contract")
    return y


def fpq_conv2d_quantize_input(x, x_scale, fx: Format, fw: Format, C_out, R, S, pad, stride, workspace):
    B, C, H, W = x.shape
    _check(lib().fpq_conv2d_quantize_input(_ptr(x), float(x_scale), fx.c(), fw.c(), B, C, H, W, C_out, R, S, pad,
                                           stride, _ptr(workspace), workspace.numel(), _stream()),
           "fpq_conv2d_quantize_input")
    return workspace


def fpq_conv2d_contract(workspace, w_prepared, w_scale, x_scale, fx: Format, fw: Format, bias, y, in_shape, R, S,
                        pad, stride):
    B, C, H, W = in_shape
    C_out = y.shape[1]
    _check(lib().fpq_conv2d_contract(_ptr(workspace), workspace.numel(), _ptr(w_prepared), _ptr(w_scale),
                                     float(x_scale), fx.c(), fw.c(), _ptr(bias), _ptr(y), B, C, H, W, C_out, R, S,
                                     pad, stride, _stream()), "fpq_conv2d_contract")
    return y


def fpq_linear_static(x, w_prepared, w_scale, x_scale, fx: Format, fw: Format, bias, y):
    """fpq_linear for callers that cannot supply a workspace: the activation codes go to a
    fixed STATIC_SCRATCH_BYTES array inside the library.  `y` is passed in, so the call itself
    creates no tensor and allocates nothing.  Calls must not overlap on the GPU."""
    M, K = x.shape
    N = y.shape[1]
    _check(lib().fpq_linear_static(_ptr(x), _ptr(w_prepared), _ptr(w_scale), float(x_scale), fx.c(), fw.c(),
                                   _ptr(bias), _ptr(y), M, N, K, _stream()), "fpq_linear_static")
    return y


def fpq_linear_host(x_host, x_dev, w_prepared, w_scale, x_scale, fx, fw, bias, y_dev, y_host, workspace):
    """x_host / y_host: pinned CPU tensors; x_dev / y_dev: device staging tensors."""
    M, K = x_host.shape
    N = y_host.shape[1]
    _check(lib().fpq_linear_host(_ptr(x_host), _ptr(x_dev), _ptr(w_prepared), _ptr(w_scale), float(x_scale),
                                 fx.c(), fw.c(), _ptr(bias), _ptr(y_dev), _ptr(y_host), M, N, K, _ptr(workspace),
                                 workspace.numel(), _stream()), "fpq_linear_host")
    return y_host


def fpq_conv2d_host(x_host, x_dev, w_prepared, w_scale, x_scale, fx, fw, bias, y_dev, y_host, R, S, pad, stride,
                    workspace):
    B, C, H, W = x_host.shape
    C_out = y_host.shape[1]
    _check(lib().fpq_conv2d_host(_ptr(x_host), _ptr(x_dev), _ptr(w_prepared), _ptr(w_scale), float(x_scale),
                                 fx.c(), fw.c(), _ptr(bias), _ptr(y_dev), _ptr(y_host), B, C, H, W, C_out, R, S,
                                 pad, stride, _ptr(workspace), workspace.numel(), _stream()), "fpq_conv2d_host")
    return y_host


def fpq_prepare_weight_split(codes: torch.Tensor, fmt: Format, N: int, C1: int, C2: int, R: int, S: int) -> torch.Tensor:
    """Contraction-ready weights of a convolution over two concatenated input tensors."""
    size = lib().fpq_prepared_size_split(fmt.c(), N, C1, C2, R, S)
    assert size > 0, "invalid split layer"
    prepared = torch.empty(size, dtype=torch.uint8, device=codes.device)
    _check(lib().fpq_prepare_weight_split(_ptr(codes), fmt.c(), N, C1, C2, R, S, _ptr(prepared), _stream()),
           "fpq_prepare_weight_split")
    return prepared


def fpq_conv2d_split_workspace_size(B, C1, C2, H, W, C_out, R, S, pad, stride, fx: Format, fw: Format) -> int:
    return lib().fpq_conv2d_split_workspace_size(B, C1, C2, H, W, C_out, R, S, pad, stride, fx.c(), fw.c())


def fpq_conv2d_split(x1, x1_scale, x2, x2_scale, w_prepared, w_scale, fx: Format, fw: Format, bias, y, R, S, pad,
                     stride, workspace):
    """Convolution over the channel concatenation of x1 and x2, quantized with their own scales."""
    B, C1, H, W = x1.shape
    C2 = x2.shape[1]
    C_out = y.shape[1]
    _check(lib().fpq_conv2d_split(_ptr(x1), C1, float(x1_scale), _ptr(x2), C2, float(x2_scale), _ptr(w_prepared),
                                  _ptr(w_scale), fx.c(), fw.c(), _ptr(bias), _ptr(y), B, H, W, C_out, R, S, pad, stride,
                                  _ptr(workspace), workspace.numel(), _stream()), "fpq_conv2d_split")
    return y


def fpq_zero_census(codes: torch.Tensor, n: int, fmt: Format, count: torch.Tensor = None) -> torch.Tensor:
    """Number of zero codes among the n values of `codes` (device int64 tensor with one entry)."""
    assert codes.is_cuda and codes.dtype == torch.uint8 and codes.is_contiguous()
    if count is None:
        count = torch.empty(1, dtype=torch.int64, device=codes.device)
    _check(lib().fpq_zero_census(_ptr(codes), int(n), fmt.c(), _ptr(count), _stream()), "fpq_zero_census")
    return count


def fpq_search_workspace_size(n_enc: int, n_clip: int) -> int:
    return lib().fpq_search_workspace_size(int(n_enc), int(n_clip))


def fpq_search_clip_candidates(maxabs: float, count: int = 111) -> torch.Tensor:
    """The evenly spaced clipping candidates up to maxabs, as a CPU float32 tensor."""
    out = torch.empty(count, dtype=torch.float32)
    _check(lib().fpq_search_clip_candidates(float(maxabs), int(count), ctypes.c_void_p(out.data_ptr())),
           "fpq_search_clip_candidates")
    return out


def fpq_search_format(x: torch.Tensor, encodings, clip: torch.Tensor, mse: torch.Tensor = None,
                      best: torch.Tensor = None, workspace: torch.Tensor = None):
    """Mean squared error of every (encoding, clipping value) candidate on x and Algorithm 1's
    choice.  Returns (mse [n_enc][n_clip] float64, best [2] int32), both on the device."""
    assert x.is_cuda and x.dtype == torch.float32 and x.is_contiguous()
    assert clip.is_cuda and clip.dtype == torch.float32 and clip.is_contiguous()
    n_enc, n_clip = len(encodings), clip.numel()
    enc = (_CFormat * n_enc)(*[f.c() for f in encodings])
    if mse is None:
        mse = torch.empty((n_enc, n_clip), dtype=torch.float64, device=x.device)
    if best is None:
        best = torch.empty(2, dtype=torch.int32, device=x.device)
    if workspace is None:
        workspace = torch.empty(max(8, fpq_search_workspace_size(n_enc, n_clip)), dtype=torch.uint8, device=x.device)
    _check(lib().fpq_search_format(_ptr(x), x.numel(), ctypes.cast(enc, ctypes.c_void_p), n_enc, _ptr(clip), n_clip,
                                   _ptr(mse), _ptr(best), _ptr(workspace), workspace.numel(), _stream()),
           "fpq_search_format")
    return mse, best


def fpq_round_learn_workspace_size(M: int, N: int, K: int) -> int:
    return lib().fpq_round_learn_workspace_size(int(M), int(N), int(K))


def fpq_round_learn_step(w: torch.Tensor, scale: torch.Tensor, fmt: Format, alpha: torch.Tensor, a: torch.Tensor,
                         reg: float, lr: float = 0.0, grad: torch.Tensor = None, loss: torch.Tensor = None,
                         workspace: torch.Tensor = None):
    """One evaluation of the rounding-learning objective and its gradient (Sec. V-B); alpha is updated in
    place when lr != 0.  Returns (grad [N][K] float32, loss [2] float64 = {mse, sum of lambda}), on the device."""
    for t_ in (w, scale, alpha, a):
        assert t_.is_cuda and t_.dtype == torch.float32 and t_.is_contiguous()
    N, K = w.shape
    M = a.shape[0]
    assert a.shape == (M, K) and alpha.shape == (N, K) and scale.shape == (N,)
    if grad is None:
        grad = torch.empty((N, K), dtype=torch.float32, device=w.device)
    if loss is None:
        loss = torch.empty(2, dtype=torch.float64, device=w.device)
    if workspace is None:
        workspace = torch.empty(max(256, fpq_round_learn_workspace_size(M, N, K)), dtype=torch.uint8, device=w.device)
    _check(lib().fpq_round_learn_step(_ptr(w), _ptr(scale), fmt.c(), _ptr(alpha), _ptr(a), M, N, K, float(reg),
                                      float(lr), _ptr(grad), _ptr(loss), _ptr(workspace), workspace.numel(),
                                      _stream()), "fpq_round_learn_step")
    return grad, loss


def fpq_round_learn_unfold(x: torch.Tensor, R: int, S: int, pad: int, stride: int, rows: torch.Tensor = None) -> torch.Tensor:
    """Input rows [B*H_out*W_out][C*R*S] of a convolution over x (NCHW), columns in [C][R][S] order."""
    assert x.is_cuda and x.dtype == torch.float32 and x.is_contiguous() and x.dim() == 4
    B, C, H, W = x.shape
    Ho, Wo = (H + 2 * pad - R) // stride + 1, (W + 2 * pad - S) // stride + 1
    if rows is None:
        rows = torch.empty((B * Ho * Wo, C * R * S), dtype=torch.float32, device=x.device)
    _check(lib().fpq_round_learn_unfold(_ptr(x), B, C, H, W, R, S, pad, stride, _ptr(rows), _stream()),
           "fpq_round_learn_unfold")
    return rows


def fpq_round_learn_harden(alpha: torch.Tensor, bits: torch.Tensor = None) -> torch.Tensor:
    """Decision bits (alpha >= 0) packed as fpq_quantize_weight reads them: [N][ceil(K/8)] bytes."""
    assert alpha.is_cuda and alpha.dtype == torch.float32 and alpha.is_contiguous() and alpha.dim() == 2
    N, K = alpha.shape
    if bits is None:
        bits = torch.empty((N, (K + 7) // 8), dtype=torch.uint8, device=alpha.device)
    _check(lib().fpq_round_learn_harden(_ptr(alpha), N, K, _ptr(bits), _stream()), "fpq_round_learn_harden")
    return bits


def fpq_set_path_policy(policy: int) -> None:
    _check(lib().fpq_set_path_policy(int(policy)), "fpq_set_path_policy")


def fpq_get_path_policy() -> int:
    return lib().fpq_get_path_policy()


def fpq_selftest_bounded_wait(limit_cycles: int) -> None:
    """One warp waits limit_cycles on a barrier nobody arrives on, then records ERR_TIMEOUT in the status word."""
    _check(lib().fpq_selftest_bounded_wait(int(limit_cycles), _stream()), "fpq_selftest_bounded_wait")


def fpq_conv2d_route(B, C, H, W, C_out, R, S, pad, stride, fx: Format, fw: Format) -> int:
    """Which kernels fpq_conv2d would run for this shape under the current policy (ROUTE_*)."""
    r = lib().fpq_conv2d_route(B, C, H, W, C_out, R, S, pad, stride, fx.c(), fw.c())
    if r < 0:
        _check(r, "fpq_conv2d_route")
    return r


def fpq_read_status() -> int:
    return lib().fpq_read_status(_stream())
