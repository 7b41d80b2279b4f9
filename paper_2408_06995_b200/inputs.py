"""Seeded synthetic inputs shaped like the paper's U-Net layers.

This module holds no quantization arithmetic: it only draws FP32 tensors
(activations, weights, biases, rounding decisions) with the shapes and value
distributions of the workloads, so that the CUDA library and an independent
checker can be fed identical bytes.  The paper's own workloads are DDIM on
CIFAR-10, LDM-4 on LSUN-Bedroom and Stable Diffusion v1.5 / SDXL (Sec. VI-A);
their checkpoints and calibration data are replaced by random draws of the same
shapes.  Tensor j of workload i uses seed 1000*i + j.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np


def _rng(workload: int, tensor: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(1000 * workload + tensor))


def _normal(rng, shape, std=1.0):
    return (rng.standard_normal(shape, dtype=np.float32) * np.float32(std)).astype(np.float32)


def _with_outliers(rng, x, frac, factor):
    n = x.size
    k = max(1, int(round(n * frac)))
    pos = rng.choice(n, size=k, replace=False)
    flat = x.reshape(-1)
    flat[pos] *= np.float32(factor)
    return x


def _per_channel(rng, w):
    u = rng.uniform(0.5, 2.0, size=w.shape[0]).astype(np.float32)
    return (w * u.reshape((-1,) + (1,) * (w.ndim - 1))).astype(np.float32)


def _silu(x):
    return (x / (1.0 + np.exp(-x.astype(np.float64)))).astype(np.float32)


def _student_t4(rng, shape):
    z = rng.standard_normal(shape, dtype=np.float32).astype(np.float64)
    chi2 = (rng.standard_normal((4,) + tuple(shape), dtype=np.float32).astype(np.float64) ** 2).sum(0)
    return (z / np.sqrt(chi2 / 4.0)).astype(np.float32)


def bernoulli_bits(rng, N, K):
    """Stand-in for hardened learned rounding decisions: [N][K] of 0/1, p = 0.5."""
    return rng.integers(0, 2, size=(N, K), dtype=np.uint8)


@dataclass
class Layer:
    """One quantized layer of a workload (shapes only unless tensors are drawn)."""

    name: str
    kind: str                      # "linear" or "conv"
    M: int = 0                     # linear rows / conv B*Ho*Wo
    N: int = 0                     # out features / out channels
    K: int = 0                     # in features / C*R*S
    B: int = 0
    C: int = 0
    H: int = 0
    W: int = 0
    R: int = 1
    S: int = 1
    pad: int = 0
    stride: int = 1
    wfmt: str = "e4m3"             # "e4m3" or "e2m1"
    rounding: bool = False         # learned-rounding decisions supplied
    count: int = 1                 # how many times the shape occurs in a trace
    x: Optional[np.ndarray] = None
    w: Optional[np.ndarray] = None
    bias: Optional[np.ndarray] = None
    bits: Optional[np.ndarray] = None   # [N][K] 0/1

    @property
    def Ho(self):
        return (self.H + 2 * self.pad - self.R) // self.stride + 1

    @property
    def Wo(self):
        return (self.W + 2 * self.pad - self.S) // self.stride + 1

    @property
    def flops(self):
        return 2 * self.M * self.N * self.K


def linear_layer(name, M, K, N, wfmt="e4m3", rounding=False, count=1) -> Layer:
    return Layer(name=name, kind="linear", M=M, N=N, K=K, wfmt=wfmt, rounding=rounding, count=count)


def conv_layer(name, B, C, H, W, Co, R, pad=None, stride=1, wfmt="e4m3", rounding=False, count=1) -> Layer:
    pad = (R // 2) if pad is None else pad
    L = Layer(name=name, kind="conv", B=B, C=C, H=H, W=W, N=Co, R=R, S=R, pad=pad, stride=stride,
              wfmt=wfmt, rounding=rounding, count=count)
    L.K = C * R * R
    L.M = B * L.Ho * L.Wo
    return L


def draw(layer: Layer, workload: int, tensor0: int = 0, x_law="normal", w_std=0.02,
         per_channel=False, bias_std=0.01, outlier=None) -> Layer:
    """Fill a layer's tensors.  x_law: normal | silu | t4 (Student-t, 4 dof, x0.5)."""
    r_x, r_w, r_b, r_h, r_o = (_rng(workload, tensor0 + j) for j in range(5))
    xshape = (layer.M, layer.K) if layer.kind == "linear" else (layer.B, layer.C, layer.H, layer.W)
    wshape = (layer.N, layer.K) if layer.kind == "linear" else (layer.N, layer.C, layer.R, layer.S)
    if x_law == "normal":
        x = _normal(r_x, xshape)
    elif x_law == "silu":
        x = _silu(_normal(r_x, xshape))
    elif x_law == "t4":
        x = (_student_t4(r_x, xshape) * np.float32(0.5)).astype(np.float32)
    else:
        raise ValueError(x_law)
    if outlier is not None:
        x = _with_outliers(r_o, x, outlier[0], outlier[1])
    w = _normal(r_w, wshape, w_std)
    if per_channel:
        w = _per_channel(r_w, w)
    layer.x = np.ascontiguousarray(x)
    layer.w = np.ascontiguousarray(w)
    layer.bias = _normal(r_b, (layer.N,), bias_std)
    layer.bits = bernoulli_bits(r_h, layer.N, layer.K) if layer.rounding else None
    return layer


# ---- the five workloads ------------------------------------------------------

def config1() -> List[Layer]:
    """Single W8A8 linear: X [256,512] ~ N(0,1) with 0.1 % of entries x20,
    W [512,512] ~ N(0,0.02) x per-row U[0.5,2], bias ~ N(0,0.01)."""
    L = linear_layer("linear_256x512x512", 256, 512, 512, "e4m3")
    return [draw(L, 1, 0, "normal", 0.02, True, 0.01, (0.001, 20.0))]


def config2(batch: int = 64) -> List[Layer]:
    """DDIM-CIFAR-style 3x3 conv, W8A8 with rounding decisions: X [64,128,32,32] =
    SiLU(N(0,1)), W [128,128,3,3] ~ N(0,0.03) per-channel scaled."""
    L = conv_layer("conv3x3_128_128_32", batch, 128, 32, 32, 128, 3, wfmt="e4m3", rounding=True)
    return [draw(L, 2, 0, "silu", 0.03, True)]


def config3(batch: int = 16) -> List[Layer]:
    """LDM-4-style pair, W4A8: conv3x3 256->256 and conv1x1 256->512 at 32x32,
    activations 0.5 * Student-t(4), weights N(0,0.02), Bernoulli rounding bits."""
    a = conv_layer("conv3x3_256_256_32", batch, 256, 32, 32, 256, 3, wfmt="e2m1", rounding=True)
    b = conv_layer("conv1x1_256_512_32", batch, 256, 32, 32, 512, 1, wfmt="e2m1", rounding=True)
    return [draw(a, 3, 0, "t4", 0.02), draw(b, 3, 10, "t4", 0.02)]


def config4(M: int = 8192) -> List[Layer]:
    """SD-v1 transformer-block linears at 64x64 latent, batch 2, in W8A8 and W4A8."""
    out = []
    shapes = [("qkv", 320, 960), ("attn_out", 320, 320), ("geglu", 320, 2560), ("ffn_out", 1280, 320)]
    t = 0
    for wf in ("e4m3", "e2m1"):
        for nm, K, N in shapes:
            L = linear_layer(f"{nm}_{K}_{N}_{wf}", M, K, N, wf, rounding=(wf == "e2m1"))
            out.append(draw(L, 4, t, "normal", 0.02, False, 0.01, (0.0005, 30.0)))
            t += 10
    return out


def sd_v1_unet_layers(batch: int = 2, latent: int = 64, wfmt: str = "e2m1") -> List[Layer]:
    """Every conv and linear of one denoising step of an SD-v1-style U-Net
    (base width 320, multipliers 1/2/4/4, two residual blocks per level,
    transformer blocks at the three highest resolutions and in the middle,
    77 text tokens of width 768), in execution order, shapes only."""
    Ls: List[Layer] = []
    ch, temb, ctx, ntok = 320, 1280, 768, 77
    rd = wfmt == "e2m1"

    def conv(name, C, res, Co, R, stride=1):
        Ls.append(conv_layer(name, batch, C, res, res, Co, R, stride=stride, wfmt=wfmt, rounding=rd))

    def lin(name, M, K, N):
        Ls.append(linear_layer(name, M, K, N, wfmt, rounding=rd))

    def res_block(tag, cin, cout, res):
        conv(f"{tag}.conv1", cin, res, cout, 3)
        lin(f"{tag}.temb", batch, temb, cout)
        conv(f"{tag}.conv2", cout, res, cout, 3)
        if cin != cout:
            conv(f"{tag}.skip", cin, res, cout, 1)

    def transformer(tag, C, res):
        T = batch * res * res
        conv(f"{tag}.proj_in", C, res, C, 1)
        lin(f"{tag}.attn1.qkv", T, C, 3 * C)
        lin(f"{tag}.attn1.out", T, C, C)
        lin(f"{tag}.attn2.q", T, C, C)
        lin(f"{tag}.attn2.kv", batch * ntok, ctx, 2 * C)
        lin(f"{tag}.attn2.out", T, C, C)
        lin(f"{tag}.ff.geglu", T, C, 8 * C)
        lin(f"{tag}.ff.out", T, 4 * C, C)
        conv(f"{tag}.proj_out", C, res, C, 1)

    lin("time.fc1", batch, ch, temb)
    lin("time.fc2", batch, temb, temb)
    conv("conv_in", 4, latent, ch, 3)
    mult = (1, 2, 4, 4)
    res = latent
    cur = ch
    skips = [ch]
    for lvl, mlt in enumerate(mult):
        cout = ch * mlt
        for i in range(2):
            res_block(f"down{lvl}.res{i}", cur, cout, res)
            cur = cout
            if lvl < 3:
                transformer(f"down{lvl}.attn{i}", cur, res)
            skips.append(cur)
        if lvl < 3:
            conv(f"down{lvl}.downsample", cur, res, cur, 3, stride=2)
            res //= 2
            skips.append(cur)
    res_block("mid.res0", cur, cur, res)
    transformer("mid.attn", cur, res)
    res_block("mid.res1", cur, cur, res)
    for lvl in (3, 2, 1, 0):
        cout = ch * mult[lvl]
        for i in range(3):
            cin = cur + skips.pop()
            res_block(f"up{lvl}.res{i}", cin, cout, res)
            cur = cout
            if lvl < 3:
                transformer(f"up{lvl}.attn{i}", cur, res)
        if lvl > 0:
            res *= 2
            conv(f"up{lvl}.upsample", cur, res, cur, 3)
    conv("conv_out", ch, latent, 4, 3)
    return Ls


def distinct_shapes(layers: List[Layer]) -> List[Layer]:
    """Collapse a trace to its distinct shapes, with occurrence counts."""
    seen = {}
    for L in layers:
        key = (L.kind, L.M, L.N, L.K, L.B, L.C, L.H, L.W, L.R, L.pad, L.stride, L.wfmt)
        if key in seen:
            seen[key].count += 1
        else:
            import copy
            c = copy.copy(L)
            c.count = 1
            seen[key] = c
    return list(seen.values())
