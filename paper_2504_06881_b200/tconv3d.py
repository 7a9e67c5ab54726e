"""Thin ctypes binding over the three-dimensional entry points of libtconv.so (include/tconv3d.h).

Argument marshalling only; every step runs in the library's CUDA kernels.  A layer is described
by a dict with N, C, D, H, W, K, T, R, S, the triples ``stride`` / ``pad`` / ``dil`` in
(depth, height, width) order, and ``mode`` / ``chan`` / ``dtype`` by name.
"""
from __future__ import annotations

import ctypes

import torch

from .tconv import CHANS, DTYPES, MODES, TORCH_DTYPE, TconvError, _check, _lib, _on_stream, _p, _stream

# every symbol include/tconv3d.h declares
SYMBOLS = ("tconv3d_output_shape", "tconv3d_winner_bytes", "tconv3d_workspace_bytes", "tconv3d_forward",
           "tconv3d_backward", "tconv3d_launch_count")


class Desc3(ctypes.Structure):
    """tconv3d_desc_t."""
    _fields_ = [(n, ctypes.c_int32) for n in (
        "N", "C", "D", "H", "W", "K", "T", "R", "S", "stride_d", "stride_h", "stride_w", "pad_d", "pad_h",
        "pad_w", "dil_d", "dil_h", "dil_w", "mode", "chan", "dtype")]


def _bind():
    vp, fp, sz = ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t
    dp, ip = ctypes.POINTER(Desc3), ctypes.POINTER(ctypes.c_int32)
    _lib.tconv3d_output_shape.argtypes = [dp, ip, ip, ip]
    _lib.tconv3d_output_shape.restype = ctypes.c_int
    _lib.tconv3d_winner_bytes.argtypes = [dp]
    _lib.tconv3d_winner_bytes.restype = sz
    _lib.tconv3d_workspace_bytes.argtypes = [dp, ctypes.c_int]
    _lib.tconv3d_workspace_bytes.restype = sz
    _lib.tconv3d_forward.argtypes = [dp, vp, vp, vp, fp, fp, fp, vp, vp, vp]
    _lib.tconv3d_forward.restype = ctypes.c_int
    _lib.tconv3d_backward.argtypes = [dp, vp, vp, vp, fp, fp, vp, vp, vp, fp, fp, fp, fp, fp, vp, sz, vp]
    _lib.tconv3d_backward.restype = ctypes.c_int
    _lib.tconv3d_launch_count.restype = ctypes.c_longlong


_bind()


def make_desc(d: dict) -> Desc3:
    return Desc3(*(d[k] for k in "NCDHWKTRS"), *d["stride"], *d["pad"], *d["dil"], MODES[d["mode"]],
                 CHANS[d.get("chan", "default")], DTYPES[d.get("dtype", "f32")])


# ---- the C entry points, one to one ------------------------------------------------
def tconv3d_output_shape(d: dict):
    od, oh, ow = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()
    rc = _lib.tconv3d_output_shape(ctypes.byref(make_desc(d)), ctypes.byref(od), ctypes.byref(oh),
                                   ctypes.byref(ow))
    if rc != 0:
        raise TconvError(rc, "tconv3d_output_shape")
    return od.value, oh.value, ow.value


def tconv3d_winner_bytes(d: dict) -> int:
    return int(_lib.tconv3d_winner_bytes(ctypes.byref(make_desc(d))))


def tconv3d_workspace_bytes(d: dict, backward: bool) -> int:
    return int(_lib.tconv3d_workspace_bytes(ctypes.byref(make_desc(d)), int(backward)))


def tconv3d_forward(d: dict, x, w, w2, alpha, beta, bias, y, winners=None, stream=None) -> int:
    return _lib.tconv3d_forward(ctypes.byref(make_desc(d)), _p(x), _p(w), _p(w2), _p(alpha), _p(beta),
                                _p(bias), _p(y), _p(winners), _stream(stream))


def tconv3d_backward(d: dict, x, w, w2, alpha, beta, grad_y, winners, grad_x, grad_w, grad_w2, grad_alpha,
                     grad_beta, grad_bias, workspace, stream=None) -> int:
    nbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    return _lib.tconv3d_backward(ctypes.byref(make_desc(d)), _p(x), _p(w), _p(w2), _p(alpha), _p(beta),
                                 _p(grad_y), _p(winners), _p(grad_x), _p(grad_w), _p(grad_w2),
                                 _p(grad_alpha), _p(grad_beta), _p(grad_bias), _p(workspace), nbytes,
                                 _stream(stream))


def tconv3d_launch_count() -> int:
    return int(_lib.tconv3d_launch_count())


# ---- allocation helpers -------------------------------------------------------------
def _shapes(d):
    N, C, D, H, W, K, T, R, S = (d[k] for k in "NCDHWKTRS")
    return (N, C, D, H, W), (K, C, T, R, S), (N, K) + tconv3d_output_shape(d)


def winner_buffer(d: dict, device):
    """Buffer for the winning taps: uint16 [N,K,C,OD,OH,OW] (Sum channel combine) or int32 [N,K,OD,OH,OW]."""
    _, _, sy = _shapes(d)
    chan = d.get("chan", "default")
    if chan == "default":
        chan = {"max_plus": "max", "min_plus": "min"}.get(d["mode"], "sum")
    if chan == "sum":
        return torch.empty((sy[0], sy[1], d["C"]) + sy[2:], dtype=torch.int16, device=device)
    return torch.empty(sy, dtype=torch.int32, device=device)


def forward(d: dict, x, w, w2=None, alpha=None, beta=None, bias=None, want_winners=False, stream=None):
    """Allocate y (and the winners) and run tconv3d_forward.  Returns (y, winners)."""
    sx, sw, sy = _shapes(d)
    dt = TORCH_DTYPE[d.get("dtype", "f32")]
    _check(x, sx, dt, "x"); _check(w, sw, dt, "w"); _check(w2, sw, dt, "w2")
    _check(alpha, (d["K"], d["C"]), torch.float32, "alpha"); _check(beta, (d["K"], d["C"]), torch.float32, "beta")
    _check(bias, (d["K"],), torch.float32, "bias")
    y = torch.empty(sy, dtype=dt, device=x.device)
    winners = winner_buffer(d, x.device) if want_winners else None
    _on_stream(stream, y, winners)
    rc = tconv3d_forward(d, x, w, w2, alpha, beta, bias, y, winners, stream)
    if rc != 0:
        raise TconvError(rc, "tconv3d_forward")
    return y, winners


def backward(d: dict, x, w, grad_y, w2=None, alpha=None, beta=None, winners=None, need_grad_x=True,
             stream=None):
    """Allocate every gradient the mode has and run tconv3d_backward.  Returns a dict."""
    sx, sw, sy = _shapes(d)
    dt = TORCH_DTYPE[d.get("dtype", "f32")]
    _check(x, sx, dt, "x"); _check(w, sw, dt, "w"); _check(w2, sw, dt, "w2"); _check(grad_y, sy, dt, "grad_y")
    two, par = d["mode"] in ("compound", "parallel"), d["mode"] == "parallel"
    dev, f32 = x.device, torch.float32
    out = {"grad_w": torch.empty(sw, dtype=f32, device=dev), "grad_bias": torch.empty((d["K"],), dtype=f32, device=dev)}
    if need_grad_x:
        out["grad_x"] = torch.empty(sx, dtype=dt, device=dev)
    if par:
        out["grad_w2"] = torch.empty(sw, dtype=f32, device=dev)
    if two:
        out["grad_alpha"] = torch.empty((d["K"], d["C"]), dtype=f32, device=dev)
        out["grad_beta"] = torch.empty((d["K"], d["C"]), dtype=f32, device=dev)
    ws = torch.empty(tconv3d_workspace_bytes(d, True), dtype=torch.uint8, device=dev)
    _on_stream(stream, ws, *out.values())
    rc = tconv3d_backward(d, x, w, w2, alpha, beta, grad_y, winners, out.get("grad_x"), out["grad_w"],
                          out.get("grad_w2"), out.get("grad_alpha"), out.get("grad_beta"), out["grad_bias"],
                          ws, stream)
    if rc != 0:
        raise TconvError(rc, "tconv3d_backward")
    return out
