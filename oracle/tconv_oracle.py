"""ctypes front end of the CPU oracle (test infrastructure, NOT a product path).

Only tests, the smoke check and the benchmark's CPU-baseline leg may use this
module.  It compiles ``tconv_oracle.c`` (plain C, OpenMP over outputs) with gcc
next to the source and exposes the forward pass, the backward pass and the
operation tallies of the paper's Section 4.1.  It imports nothing from the CUDA
package.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "tconv_oracle.c"
_LIB = _HERE / "libtconv_oracle.so"

MODES = {"max_plus": 0, "min_plus": 1, "compound": 2, "parallel": 3}
CHANS = {"default": 0, "sum": 1, "max": 2, "min": 3}
DTYPES = {"f32": 0, "bf16": 1}
PAD_MODES = {"zero": 0, "neutral": 1}


class _Desc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "N", "C", "H", "W", "K", "R", "S", "stride_h", "stride_w", "pad_h", "pad_w",
        "dil_h", "dil_w", "mode", "chan", "dtype", "pad_mode")]


class _Counts(ctypes.Structure):
    _fields_ = [("adds", ctypes.c_int64), ("cmps", ctypes.c_int64), ("muls", ctypes.c_int64)]


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc if the library is missing or older than its source."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".{os.getpid()}.tmp.so")
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               "-fno-fast-math", str(_SRC), "-o", str(tmp), "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(str(_LIB))
        _lib.ora_threads.restype = ctypes.c_int
        _lib.ora_forward.restype = ctypes.c_int
        _lib.ora_backward.restype = ctypes.c_int
    return _lib


def threads() -> int:
    """Number of OpenMP threads the oracle will use."""
    return int(_load().ora_threads())


def make_desc(N, C, H, W, K, R, S, stride=(1, 1), pad=(0, 0), dil=(1, 1),
              mode="max_plus", chan="default", dtype="f32") -> dict:
    return dict(N=N, C=C, H=H, W=W, K=K, R=R, S=S, stride_h=stride[0], stride_w=stride[1],
                pad_h=pad[0], pad_w=pad[1], dil_h=dil[0], dil_w=dil[1],
                mode=mode, chan=chan, dtype=dtype)


def _cdesc(d: dict) -> _Desc:
    return _Desc(d["N"], d["C"], d["H"], d["W"], d["K"], d["R"], d["S"], d["stride_h"],
                 d["stride_w"], d["pad_h"], d["pad_w"], d["dil_h"], d["dil_w"],
                 MODES[d["mode"]], CHANS[d["chan"]], DTYPES[d["dtype"]],
                 PAD_MODES[d.get("pad_mode", "zero")])


def output_shape(d: dict):
    def ext(i, p, dl, k, s):
        span = i + 2 * p - dl * (k - 1) - 1
        return 0 if span < 0 else span // s + 1
    return (ext(d["H"], d["pad_h"], d["dil_h"], d["R"], d["stride_h"]),
            ext(d["W"], d["pad_w"], d["dil_w"], d["S"], d["stride_w"]))


def resolved_chan(d: dict) -> str:
    if d["chan"] != "default":
        return d["chan"]
    return {"max_plus": "max", "min_plus": "min"}.get(d["mode"], "sum")


def _f32(a, shape=None):
    if a is None:
        return None
    a = np.ascontiguousarray(a, dtype=np.float32)
    if shape is not None:
        assert a.shape == tuple(shape), (a.shape, shape)
    return a


def _ptr(a, ctype=ctypes.c_float):
    if a is None:
        return None
    return a.ctypes.data_as(ctypes.POINTER(ctype))


def _is_bf16(a) -> bool:
    if a is None:
        return True
    bits = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    return bool(np.all((bits & 0xFFFF) == 0))


def forward(d: dict, x, w, w2=None, alpha=None, beta=None, bias=None,
            want_winners: bool = True, want_counts: bool = False):
    """Run the oracle forward.  Returns a dict with ``y`` and, on request,
    ``idx`` (int32 [N,K,OH,OW], Max/Min channel combine), ``codes`` (uint8
    [N,K,C,OH,OW], Sum channel combine, only if R*S <= 16) and ``counts``."""
    lib = _load()
    OH, OW = output_shape(d)
    N, C, H, W, K, R, S = (d[k] for k in "NCHWKRS")
    x = _f32(x, (N, C, H, W)); w = _f32(w, (K, C, R, S)); w2 = _f32(w2, (K, C, R, S))
    alpha = _f32(alpha, (K, C)); beta = _f32(beta, (K, C)); bias = _f32(bias, (K,))
    if d["dtype"] == "bf16":
        assert _is_bf16(x) and _is_bf16(w) and _is_bf16(w2), "bf16 mode needs bf16-valued inputs"
    y = np.empty((N, K, OH, OW), np.float32)
    chan = resolved_chan(d)
    idx = codes = None
    if want_winners and chan != "sum":
        idx = np.full((N, K, OH, OW), -1, np.int32)
    if want_winners and chan == "sum" and R * S <= 16:
        codes = np.zeros((N, K, C, OH, OW), np.uint8)
    cnt = _Counts() if want_counts else None
    rc = lib.ora_forward(ctypes.byref(_cdesc(d)), _ptr(x), _ptr(w), _ptr(w2), _ptr(alpha),
                         _ptr(beta), _ptr(bias), _ptr(y), _ptr(idx, ctypes.c_int32),
                         _ptr(codes, ctypes.c_uint8),
                         ctypes.byref(cnt) if cnt is not None else None)
    if rc != 0:
        raise ValueError(f"oracle forward rejected the descriptor (rc={rc})")
    out = {"y": y, "idx": idx, "codes": codes}
    if cnt is not None:
        out["counts"] = {"adds": cnt.adds, "cmps": cnt.cmps, "muls": cnt.muls}
    return out


def channel_stats(y):
    """Per-channel sums of an output y[N][K][OH][OW] and of its squares, in float64, with the sums
    of absolute values beside them (the scale of a summation error bound): what the batch
    normalisation after a tropical layer (the paper's section "ResNet Models") takes its mean and
    variance from.  Returns {"sum_y": (s, abs), "sum_y2": (s, abs)}."""
    y = np.asarray(y, np.float64)
    return {"sum_y": (y.sum(axis=(0, 2, 3)), np.abs(y).sum(axis=(0, 2, 3))),
            "sum_y2": ((y * y).sum(axis=(0, 2, 3)), (y * y).sum(axis=(0, 2, 3)))}


def backward(d: dict, x, w, g, w2=None, alpha=None, beta=None):
    """Run the oracle backward.  Returns a dict name -> (grad, abs_sum), both
    float64: ``grad_x``, ``grad_w``, ``grad_w2`` (parallel only), ``grad_alpha``,
    ``grad_beta`` (compound / parallel only), ``grad_bias``."""
    lib = _load()
    OH, OW = output_shape(d)
    N, C, H, W, K, R, S = (d[k] for k in "NCHWKRS")
    x = _f32(x, (N, C, H, W)); w = _f32(w, (K, C, R, S)); w2 = _f32(w2, (K, C, R, S))
    alpha = _f32(alpha, (K, C)); beta = _f32(beta, (K, C)); g = _f32(g, (N, K, OH, OW))
    two = d["mode"] in ("compound", "parallel")

    def pair(shape, on=True):
        if not on:
            return None, None
        return np.zeros(shape, np.float64), np.zeros(shape, np.float64)

    gx, gxa = pair((N, C, H, W)); gw, gwa = pair((K, C, R, S))
    gw2, gw2a = pair((K, C, R, S), d["mode"] == "parallel")
    ga, gaa = pair((K, C), two); gb, gba = pair((K, C), two); gbi, gbia = pair((K,))
    dp = lambda a: _ptr(a, ctypes.c_double)
    rc = lib.ora_backward(ctypes.byref(_cdesc(d)), _ptr(x), _ptr(w), _ptr(w2), _ptr(alpha),
                          _ptr(beta), _ptr(g), dp(gx), dp(gxa), dp(gw), dp(gwa), dp(gw2),
                          dp(gw2a), dp(ga), dp(gaa), dp(gb), dp(gba), dp(gbi), dp(gbia))
    if rc != 0:
        raise ValueError(f"oracle backward rejected the descriptor (rc={rc})")
    out = {"grad_x": (gx, gxa), "grad_w": (gw, gwa), "grad_bias": (gbi, gbia)}
    if d["mode"] == "parallel":
        out["grad_w2"] = (gw2, gw2a)
    if two:
        out["grad_alpha"] = (ga, gaa)
        out["grad_beta"] = (gb, gba)
    return out


# ---------------------------------------------------------------------------------------------
# Depthwise form (groups = C; the MobileNetV2 variants of the paper's Section 6 replace the
# depthwise convolutions): channel c is its own group, i.e. the dense operator above with one
# input and one output channel, applied channel by channel.  Nothing new is computed here: every
# number comes from ``forward`` / ``backward``.  Shapes: w, w2 [C][R][S]; alpha, beta, bias [C];
# y, g [N][C][OH][OW]; codes uint8 [N][C][OH][OW] (low nibble argmin tap, high nibble argmax tap).
def _dw_desc(d: dict) -> dict:
    assert d["K"] == d["C"], "depthwise: one output channel per input channel"
    return dict(d, C=1, K=1, chan="sum")


def depthwise_forward(d: dict, x, w, w2=None, alpha=None, beta=None, bias=None):
    d1 = _dw_desc(d)
    C = d["C"]
    two, par = d["mode"] in ("compound", "parallel"), d["mode"] == "parallel"
    ys, cs = [], []
    for c in range(C):
        r = forward(d1, np.ascontiguousarray(x[:, c:c + 1]), w[c][None, None],
                    w2[c][None, None] if par else None,
                    np.reshape(alpha[c], (1, 1)) if (two and alpha is not None) else None,
                    np.reshape(beta[c], (1, 1)) if (two and beta is not None) else None,
                    np.reshape(bias[c], (1,)) if bias is not None else None)
        ys.append(r["y"][:, 0])
        cs.append(None if r["codes"] is None else r["codes"][:, 0, 0])
    return {"y": np.stack(ys, 1), "codes": None if cs[0] is None else np.stack(cs, 1)}


def depthwise_backward(d: dict, x, w, g, w2=None, alpha=None, beta=None):
    """name -> (gradient, sum of |contributions|), float64; grad_w, grad_w2 [C][R][S]; the rest [C]."""
    d1 = _dw_desc(d)
    C = d["C"]
    two, par = d["mode"] in ("compound", "parallel"), d["mode"] == "parallel"
    parts = []
    for c in range(C):
        parts.append(backward(d1, np.ascontiguousarray(x[:, c:c + 1]), w[c][None, None],
                              np.ascontiguousarray(g[:, c:c + 1]), w2[c][None, None] if par else None,
                              np.reshape(alpha[c], (1, 1)) if (two and alpha is not None) else None,
                              np.reshape(beta[c], (1, 1)) if (two and beta is not None) else None))
    out = {}
    for name in parts[0]:
        if name == "grad_x":
            out[name] = tuple(np.concatenate([p[name][i] for p in parts], 1) for i in (0, 1))
        elif name in ("grad_w", "grad_w2"):
            out[name] = tuple(np.stack([p[name][i][0, 0] for p in parts], 0) for i in (0, 1))
        else:
            out[name] = tuple(np.stack([p[name][i].reshape(()) for p in parts], 0) for i in (0, 1))
    return out
