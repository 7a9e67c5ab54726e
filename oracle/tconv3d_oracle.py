"""ctypes front end of the CPU oracle for the three-dimensional tropical convolutions
(Section 3.2 and the Conv3d layers of Sections 3.4 / 3.5).  Test infrastructure, NOT a
product path: only tests, the smoke check and the benchmark's CPU-baseline leg may use it.
It compiles ``tconv3d_oracle.c`` with gcc next to the source and imports nothing from the
CUDA package.

A layer is described by a dict with N, C, D, H, W, K, T, R, S, ``stride`` / ``pad`` / ``dil``
(depth, height, width), ``mode``, ``chan``, ``dtype``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "tconv3d_oracle.c"
_LIB = _HERE / "libtconv3d_oracle.so"

MODES = {"max_plus": 0, "min_plus": 1, "compound": 2, "parallel": 3}
CHANS = {"default": 0, "sum": 1, "max": 2, "min": 3}
DTYPES = {"f32": 0, "bf16": 1}


class _Desc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in "NCDHWKTRS"] + \
               [("stride", ctypes.c_int32 * 3), ("pad", ctypes.c_int32 * 3),
                ("dil", ctypes.c_int32 * 3), ("mode", ctypes.c_int32), ("chan", ctypes.c_int32),
                ("dtype", ctypes.c_int32)]


def build(force: bool = False) -> Path:
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".{os.getpid()}.tmp.so")
        subprocess.run(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp",
                        "-ffp-contract=off", "-fno-fast-math", str(_SRC), "-o", str(tmp), "-lm"],
                       check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(str(_LIB))
    return _lib


def _cdesc(d: dict) -> _Desc:
    c = _Desc()
    for n in "NCDHWKTRS":
        setattr(c, n, int(d[n]))
    for name in ("stride", "pad", "dil"):
        getattr(c, name)[:] = [int(v) for v in d[name]]
    c.mode, c.chan, c.dtype = MODES[d["mode"]], CHANS[d.get("chan", "default")], DTYPES[d.get("dtype", "f32")]
    return c


def output_shape(d: dict):
    def ext(i, p, dl, k, s):
        span = i + 2 * p - dl * (k - 1) - 1
        return 0 if span < 0 else span // s + 1
    return tuple(ext(d[a], d["pad"][j], d["dil"][j], d[b], d["stride"][j])
                 for j, (a, b) in enumerate((("D", "T"), ("H", "R"), ("W", "S"))))


def resolved_chan(d: dict) -> str:
    ch = d.get("chan", "default")
    if ch != "default":
        return ch
    return {"max_plus": "max", "min_plus": "min"}.get(d["mode"], "sum")


def _f32(a, shape):
    if a is None:
        return None
    a = np.ascontiguousarray(a, dtype=np.float32)
    assert a.shape == tuple(shape), (a.shape, shape)
    return a


def _ptr(a, ctype=ctypes.c_float):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ctype))


def _shapes(d):
    N, C, D, H, W, K, T, R, S = (d[k] for k in "NCDHWKTRS")
    return (N, C, D, H, W), (K, C, T, R, S), (K, C), (K,), (N, K) + output_shape(d)


def forward(d: dict, x, w, w2=None, alpha=None, beta=None, bias=None):
    """``y`` float32 [N,K,OD,OH,OW]; ``idx`` int32 per output (Max / Min channel combine) or
    ``codes`` uint16 [N,K,C,OD,OH,OW] (Sum combine: argmin tap low byte, argmax tap high byte)."""
    lib = _load()
    sx, sw, sab, sb, sy = _shapes(d)
    x = _f32(x, sx); w = _f32(w, sw); w2 = _f32(w2, sw)
    alpha = _f32(alpha, sab); beta = _f32(beta, sab); bias = _f32(bias, sb)
    y = np.empty(sy, np.float32)
    idx = codes = None
    if resolved_chan(d) == "sum":
        codes = np.zeros((sy[0], sy[1], d["C"]) + sy[2:], np.uint16)
    else:
        idx = np.full(sy, -1, np.int32)
    rc = lib.o3_forward(ctypes.byref(_cdesc(d)), _ptr(x), _ptr(w), _ptr(w2), _ptr(alpha), _ptr(beta),
                        _ptr(bias), _ptr(y), _ptr(idx, ctypes.c_int32), _ptr(codes, ctypes.c_uint16))
    if rc != 0:
        raise ValueError(f"3-D oracle forward rejected the descriptor (rc={rc})")
    return {"y": y, "idx": idx, "codes": codes}


def backward(d: dict, x, w, g, w2=None, alpha=None, beta=None):
    """name -> (gradient, sum of |contributions|), both float64."""
    lib = _load()
    sx, sw, sab, sb, sy = _shapes(d)
    x = _f32(x, sx); w = _f32(w, sw); w2 = _f32(w2, sw)
    alpha = _f32(alpha, sab); beta = _f32(beta, sab); g = _f32(g, sy)
    two, par = d["mode"] in ("compound", "parallel"), d["mode"] == "parallel"

    def pair(shape, on=True):
        return (np.zeros(shape, np.float64), np.zeros(shape, np.float64)) if on else (None, None)

    gx, gw, gw2, ga, gb, gbi = pair(sx), pair(sw), pair(sw, par), pair(sab, two), pair(sab, two), pair(sb)
    dp = lambda a: _ptr(a, ctypes.c_double)
    rc = lib.o3_backward(ctypes.byref(_cdesc(d)), _ptr(x), _ptr(w), _ptr(w2), _ptr(alpha), _ptr(beta),
                         _ptr(g), dp(gx[0]), dp(gx[1]), dp(gw[0]), dp(gw[1]), dp(gw2[0]), dp(gw2[1]),
                         dp(ga[0]), dp(ga[1]), dp(gb[0]), dp(gb[1]), dp(gbi[0]), dp(gbi[1]))
    if rc != 0:
        raise ValueError(f"3-D oracle backward rejected the descriptor (rc={rc})")
    out = {"grad_x": gx, "grad_w": gw, "grad_bias": gbi}
    if par:
        out["grad_w2"] = gw2
    if two:
        out["grad_alpha"], out["grad_beta"] = ga, gb
    return out
