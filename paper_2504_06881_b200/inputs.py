"""Seeded synthetic inputs for tropical convolution layers.

This module serves both the CUDA path and the CPU checker used by the tests; it
holds none of the method's arithmetic: it only names layer geometries and draws
random tensors.  The paper's workloads are image classification (CIFAR-sized
32x32 maps, ImageNet-style 56/28/14/7 maps in a ResNet-18) and semantic
segmentation (large feature maps, atrous 3x3 convolutions); none of those
datasets is available, so tensors of the same shapes are drawn from the value
distributions a batch-normalised network produces.

Draw order is fixed: x, w, w2, alpha, beta, bias, g from one
``numpy.random.RandomState(seed)``, all as float32.  For bf16 layers x, w, w2 and
g are then rounded (nearest even) to bf16-representable float32 values.
"""
from __future__ import annotations

import numpy as np

DESC_KEYS = ("N", "C", "H", "W", "K", "R", "S", "stride_h", "stride_w", "pad_h", "pad_w",
             "dil_h", "dil_w", "mode", "chan", "dtype")


def layer(N, C, H, W, K, R=3, S=3, stride=1, pad=0, dil=1, mode="max_plus", chan="default",
          dtype="f32") -> dict:
    """Layer descriptor as a plain dict (keys = fields of the C descriptor)."""
    two = lambda v: (v, v) if isinstance(v, int) else tuple(v)
    (sh, sw), (ph, pw), (dh, dw) = two(stride), two(pad), two(dil)
    return dict(N=N, C=C, H=H, W=W, K=K, R=R, S=S, stride_h=sh, stride_w=sw, pad_h=ph,
                pad_w=pw, dil_h=dh, dil_w=dw, mode=mode, chan=chan, dtype=dtype)


def output_hw(d: dict):
    def ext(i, p, dl, k, s):
        span = i + 2 * p - dl * (k - 1) - 1
        return 0 if span < 0 else span // s + 1
    return (ext(d["H"], d["pad_h"], d["dil_h"], d["R"], d["stride_h"]),
            ext(d["W"], d["pad_w"], d["dil_w"], d["S"], d["stride_w"]))


def to_bf16_values(a: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16-representable float32 (ties to even)."""
    import torch
    return torch.from_numpy(np.ascontiguousarray(a, np.float32)).to(torch.bfloat16) \
        .to(torch.float32).numpy()


def _draw(rs, spec, shape):
    kind = spec[0]
    if kind == "normal":
        return (rs.standard_normal(shape) * spec[2] + spec[1]).astype(np.float32)
    if kind == "relu_normal":
        return np.maximum(rs.standard_normal(shape) * spec[2] + spec[1], 0).astype(np.float32)
    if kind == "uniform":
        return rs.uniform(spec[1], spec[2], shape).astype(np.float32)
    if kind == "dyadic":
        # multiples of 2^-spec[1] in [-spec[2], spec[2]]: sums of a few of them are exact
        q = 1 << spec[1]
        return (rs.randint(-spec[2] * q, spec[2] * q + 1, shape) / q).astype(np.float32)
    if kind == "ints":
        # small integers: many exact ties
        return rs.randint(spec[1], spec[2] + 1, shape).astype(np.float32)
    if kind == "const":
        return np.full(shape, spec[1], np.float32)
    raise ValueError(kind)


def draw(d: dict, seed: int, x=("normal", 0.0, 1.0), w=("normal", 0.0, 0.1),
         ab=("uniform", 0.0, 1.0), bias=("uniform", -0.1, 0.1), g=("normal", 0.0, 1.0)) -> dict:
    """Draw every tensor of one layer.  Returns float32 numpy arrays
    x[N,C,H,W], w[K,C,R,S], w2[K,C,R,S], alpha[K,C], beta[K,C], bias[K], g[N,K,OH,OW]."""
    rs = np.random.RandomState(seed)
    OH, OW = output_hw(d)
    N, C, H, W, K, R, S = (d[k] for k in "NCHWKRS")
    t = {}
    t["x"] = _draw(rs, x, (N, C, H, W))
    t["w"] = _draw(rs, w, (K, C, R, S))
    t["w2"] = _draw(rs, w, (K, C, R, S))
    t["alpha"] = _draw(rs, ab, (K, C))
    t["beta"] = _draw(rs, ab, (K, C))
    t["bias"] = _draw(rs, bias, (K,))
    t["g"] = _draw(rs, g, (N, K, OH, OW))
    if d["dtype"] == "bf16":
        for k in ("x", "w", "w2", "g"):
            t[k] = to_bf16_values(t[k])
    return t


# The five benchmark configurations (layer geometry + value distributions).
# Seeds follow 1000 + 10*cfg + variant.
def cfg1(mode="compound", chan="default"):
    d = layer(2, 3, 32, 32, 16, 3, 3, stride=1, pad=1, mode=mode, chan=chan, dtype="f32")
    return d, dict(x=("uniform", -1.0, 1.0), w=("uniform", -0.5, 0.5))


def cfg2(mode, chan="default", N=128):
    d = layer(N, 64, 32, 32, 64, 3, 3, stride=1, pad=1, mode=mode, chan=chan, dtype="f32")
    return d, dict(x=("normal", 0.0, 1.0), w=("normal", 0.0, 0.1))


def cfg3a(dtype="f32", mode="parallel", N=64):
    d = layer(N, 128, 28, 28, 128, 3, 3, stride=1, pad=1, mode=mode, dtype=dtype)
    return d, dict(x=("normal", 0.0, 1.0), w=("normal", 0.0, 0.05))


def cfg3b(dtype="f32", mode="parallel", N=64):
    d = layer(N, 64, 56, 56, 128, 3, 3, stride=2, pad=1, mode=mode, dtype=dtype)
    return d, dict(x=("normal", 0.0, 1.0), w=("normal", 0.0, 0.05))


def cfg4(dtype="bf16", mode="compound", N=8, H=128, W=256, C=256, K=256):
    d = layer(N, C, H, W, K, 3, 3, stride=1, pad=2, dil=2, mode=mode, dtype=dtype)
    return d, dict(x=("relu_normal", 0.0, 1.0), w=("normal", 0.0, 0.05))


# Three-dimensional layers (Section 3.2; the 3-D LeNet of the paper's appendix works on 28^3 and
# 64^3 volumes with 5 x 5 x 5 windows).  Descriptor keys: N, C, D, H, W, K, T, R, S and the
# triples stride / pad / dil in (depth, height, width) order.
def layer3d(N, C, D, H, W, K, T=3, R=3, S=3, stride=1, pad=0, dil=1, mode="max_plus",
            chan="default", dtype="f32") -> dict:
    three = lambda v: (v, v, v) if isinstance(v, int) else tuple(v)
    return dict(N=N, C=C, D=D, H=H, W=W, K=K, T=T, R=R, S=S, stride=three(stride), pad=three(pad),
                dil=three(dil), mode=mode, chan=chan, dtype=dtype)


def output_dhw(d: dict):
    def ext(i, p, dl, k, s):
        span = i + 2 * p - dl * (k - 1) - 1
        return 0 if span < 0 else span // s + 1
    return tuple(ext(d[a], d["pad"][j], d["dil"][j], d[b], d["stride"][j])
                 for j, (a, b) in enumerate((("D", "T"), ("H", "R"), ("W", "S"))))


def draw3d(d: dict, seed: int, x=("normal", 0.0, 1.0), w=("normal", 0.0, 0.1),
           ab=("uniform", 0.0, 1.0), bias=("uniform", -0.1, 0.1), g=("normal", 0.0, 1.0)) -> dict:
    """x[N,C,D,H,W], w / w2 [K,C,T,R,S], alpha / beta [K,C], bias[K], g[N,K,OD,OH,OW], drawn in
    that order from one ``numpy.random.RandomState(seed)``."""
    rs = np.random.RandomState(seed)
    N, C, D, H, W, K, T, R, S = (d[k] for k in "NCDHWKTRS")
    t = {}
    t["x"] = _draw(rs, x, (N, C, D, H, W))
    t["w"] = _draw(rs, w, (K, C, T, R, S))
    t["w2"] = _draw(rs, w, (K, C, T, R, S))
    t["alpha"] = _draw(rs, ab, (K, C))
    t["beta"] = _draw(rs, ab, (K, C))
    t["bias"] = _draw(rs, bias, (K,))
    t["g"] = _draw(rs, g, (N, K) + output_dhw(d))
    if d["dtype"] == "bf16":
        for k in ("x", "w", "w2", "g"):
            t[k] = to_bf16_values(t[k])
    return t
