"""Thin ctypes binding over libtconv.so (the C ABI declared in include/tconv.h).

Argument marshalling only: every step of the forward and backward passes runs in
the CUDA kernels of the library.  PyTorch supplies device memory and streams.
There is no CPU implementation here; importing this module fails loudly if the
library has not been built (``python paper_2504_06881_b200/build.py``).
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import torch

_PKG = Path(__file__).resolve().parent
LIB_PATH = _PKG / "libtconv.so"

MODES = {"max_plus": 0, "min_plus": 1, "compound": 2, "parallel": 3}
CHANS = {"default": 0, "sum": 1, "max": 2, "min": 3}
DTYPES = {"f32": 0, "bf16": 1}
PAD_MODES = {"zero": 0, "neutral": 1}
X_DTYPES = {"same": 0, "f32": 1}
TORCH_DTYPE = {"f32": torch.float32, "bf16": torch.bfloat16}

# every symbol include/tconv.h declares
SYMBOLS = ("tconv_output_shape", "tconv_winner_bytes", "tconv_workspace_bytes", "tconv_forward",
           "tconv_backward", "tconv_forward_stats", "tconv_stats_workspace_bytes", "tconv_forward_noalloc", "tconv_forward_noalloc_max_scratch", "tconv_paper_ops", "tconv_alu_probe", "tconv_alu_probe_name",
           "tconv_device_status", "tconv_status_string", "tconv_last_error", "tconv_last_kernel",
           "tconv_launch_count", "tconv_dw_winner_bytes", "tconv_dw_workspace_bytes", "tconv_dw_forward",
           "tconv_dw_backward")


class TconvError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        text = _lib.tconv_status_string(status).decode()
        detail = _lib.tconv_last_error().decode()
        super().__init__(f"{where}: {text} ({status})" + (f": {detail}" if detail else ""))


class Desc(ctypes.Structure):
    """tconv_desc_t."""
    _fields_ = [(n, ctypes.c_int32) for n in (
        "N", "C", "H", "W", "K", "R", "S", "stride_h", "stride_w", "pad_h", "pad_w",
        "dil_h", "dil_w", "mode", "chan", "dtype", "pad_mode", "x_dtype")]


def _load() -> ctypes.CDLL:
    if not LIB_PATH.exists():
        raise ImportError(f"{LIB_PATH} is missing: build it with "
                          f"`python {_PKG / 'build.py'}` (needs nvcc); there is no fallback path")
    lib = ctypes.CDLL(str(LIB_PATH))
    vp, fp, sz = ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t
    dp = ctypes.POINTER(Desc)
    lib.tconv_output_shape.argtypes = [dp, ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int32)]
    lib.tconv_output_shape.restype = ctypes.c_int
    lib.tconv_winner_bytes.argtypes = [dp]
    lib.tconv_winner_bytes.restype = sz
    lib.tconv_workspace_bytes.argtypes = [dp, ctypes.c_int]
    lib.tconv_workspace_bytes.restype = sz
    lib.tconv_forward.argtypes = [dp, vp, vp, vp, fp, fp, fp, vp, vp, vp, sz, vp]
    lib.tconv_forward.restype = ctypes.c_int
    lib.tconv_backward.argtypes = [dp, vp, vp, vp, fp, fp, vp, vp, vp, fp, fp, fp, fp, fp, vp, sz, vp]
    lib.tconv_backward.restype = ctypes.c_int
    lib.tconv_forward_stats.argtypes = [dp, vp, vp, vp, fp, fp, fp, vp, vp, fp, fp, vp, sz, vp]
    lib.tconv_forward_stats.restype = ctypes.c_int
    lib.tconv_stats_workspace_bytes.argtypes = [dp]
    lib.tconv_stats_workspace_bytes.restype = sz
    lib.tconv_forward_noalloc.argtypes = [dp, vp, vp, vp, fp, fp, fp, vp, vp, vp]
    lib.tconv_forward_noalloc.restype = ctypes.c_int
    lib.tconv_forward_noalloc_max_scratch.restype = sz
    lib.tconv_dw_winner_bytes.argtypes = [dp]
    lib.tconv_dw_winner_bytes.restype = sz
    lib.tconv_dw_workspace_bytes.argtypes = [dp, ctypes.c_int]
    lib.tconv_dw_workspace_bytes.restype = sz
    lib.tconv_dw_forward.argtypes = [dp, vp, vp, vp, fp, fp, fp, vp, vp, vp]
    lib.tconv_dw_forward.restype = ctypes.c_int
    lib.tconv_dw_backward.argtypes = [dp, vp, vp, vp, fp, fp, vp, vp, vp, fp, fp, fp, fp, fp, vp, sz, vp]
    lib.tconv_dw_backward.restype = ctypes.c_int
    lib.tconv_paper_ops.argtypes = [dp]
    lib.tconv_paper_ops.restype = ctypes.c_double
    lib.tconv_alu_probe.argtypes = [ctypes.c_int, ctypes.c_int, vp, ctypes.POINTER(ctypes.c_double), vp]
    lib.tconv_alu_probe.restype = ctypes.c_int
    lib.tconv_alu_probe_name.argtypes = [ctypes.c_int]
    lib.tconv_alu_probe_name.restype = ctypes.c_char_p
    lib.tconv_device_status.argtypes = [vp]
    lib.tconv_device_status.restype = ctypes.c_int
    lib.tconv_status_string.argtypes = [ctypes.c_int]
    lib.tconv_status_string.restype = ctypes.c_char_p
    lib.tconv_last_error.restype = ctypes.c_char_p
    lib.tconv_last_kernel.restype = ctypes.c_char_p
    lib.tconv_launch_count.restype = ctypes.c_longlong
    return lib


_lib = _load()


def make_desc(d: dict) -> Desc:
    """C descriptor from a plain dict (keys = field names; mode/chan/dtype by name)."""
    return Desc(d["N"], d["C"], d["H"], d["W"], d["K"], d["R"], d["S"], d["stride_h"],
                d["stride_w"], d["pad_h"], d["pad_w"], d["dil_h"], d["dil_w"],
                MODES[d["mode"]], CHANS[d["chan"]], DTYPES[d["dtype"]],
                PAD_MODES[d.get("pad_mode", "zero")], X_DTYPES[d.get("x_dtype", "same")])


def _p(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


# ---- the C entry points, one to one ------------------------------------------------
def tconv_output_shape(d: dict):
    oh, ow = ctypes.c_int32(), ctypes.c_int32()
    rc = _lib.tconv_output_shape(ctypes.byref(make_desc(d)), ctypes.byref(oh), ctypes.byref(ow))
    if rc != 0:
        raise TconvError(rc, "tconv_output_shape")
    return oh.value, ow.value


def tconv_winner_bytes(d: dict) -> int:
    return int(_lib.tconv_winner_bytes(ctypes.byref(make_desc(d))))


def tconv_workspace_bytes(d: dict, backward: bool) -> int:
    return int(_lib.tconv_workspace_bytes(ctypes.byref(make_desc(d)), int(backward)))


def tconv_paper_ops(d: dict) -> float:
    return float(_lib.tconv_paper_ops(ctypes.byref(make_desc(d))))


def tconv_forward(d: dict, x, w, w2, alpha, beta, bias, y, winners=None, workspace=None,
                  stream=None) -> int:
    """Raw call: tensors are passed as they are (device pointers); returns the status."""
    nbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    return _lib.tconv_forward(ctypes.byref(make_desc(d)), _p(x), _p(w), _p(w2), _p(alpha), _p(beta),
                              _p(bias), _p(y), _p(winners), _p(workspace), nbytes, _stream(stream))


def tconv_backward(d: dict, x, w, w2, alpha, beta, grad_y, winners, grad_x, grad_w, grad_w2,
                   grad_alpha, grad_beta, grad_bias, workspace=None, stream=None) -> int:
    nbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    return _lib.tconv_backward(ctypes.byref(make_desc(d)), _p(x), _p(w), _p(w2), _p(alpha),
                               _p(beta), _p(grad_y), _p(winners), _p(grad_x), _p(grad_w),
                               _p(grad_w2), _p(grad_alpha), _p(grad_beta), _p(grad_bias),
                               _p(workspace), nbytes, _stream(stream))


def tconv_forward_noalloc(d: dict, x, w, w2, alpha, beta, bias, y, winners=None, stream=None) -> int:
    """Raw call of the allocation-free forward: no workspace argument; the library's built-in
    scratch is used.  For callers that must not touch the device allocator.  Returns the status."""
    return _lib.tconv_forward_noalloc(ctypes.byref(make_desc(d)), _p(x), _p(w), _p(w2), _p(alpha),
                                      _p(beta), _p(bias), _p(y), _p(winners), _stream(stream))


def tconv_dw_winner_bytes(d: dict) -> int:
    return int(_lib.tconv_dw_winner_bytes(ctypes.byref(make_desc(d))))


def tconv_dw_workspace_bytes(d: dict, backward: bool) -> int:
    return int(_lib.tconv_dw_workspace_bytes(ctypes.byref(make_desc(d)), int(backward)))


def tconv_dw_forward(d: dict, x, w, w2, alpha, beta, bias, y, winners=None, stream=None) -> int:
    """Raw call of the depthwise forward (groups = C; d["K"] == d["C"]).  Returns the status."""
    return _lib.tconv_dw_forward(ctypes.byref(make_desc(d)), _p(x), _p(w), _p(w2), _p(alpha), _p(beta),
                                 _p(bias), _p(y), _p(winners), _stream(stream))


def tconv_dw_backward(d: dict, x, w, w2, alpha, beta, grad_y, winners, grad_x, grad_w, grad_w2,
                      grad_alpha, grad_beta, grad_bias, workspace=None, stream=None) -> int:
    nbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    return _lib.tconv_dw_backward(ctypes.byref(make_desc(d)), _p(x), _p(w), _p(w2), _p(alpha), _p(beta),
                                  _p(grad_y), _p(winners), _p(grad_x), _p(grad_w), _p(grad_w2),
                                  _p(grad_alpha), _p(grad_beta), _p(grad_bias), _p(workspace), nbytes,
                                  _stream(stream))


def tconv_stats_workspace_bytes(d: dict) -> int:
    return int(_lib.tconv_stats_workspace_bytes(ctypes.byref(make_desc(d))))


def tconv_forward_stats(d, x, w, w2, alpha, beta, bias, y, winners, sum_y, sum_y2, workspace, stream=None) -> int:
    nbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    return _lib.tconv_forward_stats(ctypes.byref(make_desc(d)), _p(x), _p(w), _p(w2), _p(alpha), _p(beta),
                                    _p(bias), _p(y), _p(winners), _p(sum_y), _p(sum_y2), _p(workspace), nbytes,
                                    _stream(stream))


def tconv_forward_noalloc_max_scratch() -> int:
    return int(_lib.tconv_forward_noalloc_max_scratch())


def tconv_alu_probe(variant: int, iters: int, sink, stream=None) -> float:
    """Launch one probe; returns the taps one launch performs."""
    taps = ctypes.c_double()
    rc = _lib.tconv_alu_probe(variant, iters, _p(sink), ctypes.byref(taps), _stream(stream))
    if rc != 0:
        raise TconvError(rc, "tconv_alu_probe")
    return taps.value


def tconv_alu_probe_name(variant: int):
    s = _lib.tconv_alu_probe_name(variant)
    return None if s is None else s.decode()


def tconv_device_status(stream=None) -> int:
    """Synchronise the stream and report (and clear) a device-side wait that gave up."""
    return _lib.tconv_device_status(_stream(stream))


def tconv_status_string(status: int) -> str:
    return _lib.tconv_status_string(status).decode()


def tconv_last_error() -> str:
    return _lib.tconv_last_error().decode()


def tconv_last_kernel() -> str:
    return _lib.tconv_last_kernel().decode()


def tconv_launch_count() -> int:
    return int(_lib.tconv_launch_count())


# ---- convenience: allocate outputs with torch, check the status ----------------------
def _check(t, shape, dtype, name):
    if t is None:
        return
    if not t.is_cuda or not t.is_contiguous() or tuple(t.shape) != tuple(shape) or t.dtype != dtype:
        raise ValueError(f"{name}: need a contiguous CUDA tensor of shape {tuple(shape)} and dtype "
                         f"{dtype}, got {tuple(t.shape)} {t.dtype} on {t.device}")


def _x_dtype(d: dict):
    """torch dtype of x: the layer's, or float32 for a bf16 layer that converts x while staging."""
    return torch.float32 if d.get("x_dtype", "same") == "f32" else TORCH_DTYPE[d["dtype"]]


def _on_stream(stream, *tensors):
    """Tensors allocated here (on the current stream) and used by kernels on `stream`: tell the
    caching allocator, so that their memory is not reused while those kernels still run."""
    if stream is None or stream == torch.cuda.current_stream():
        return
    for t in tensors:
        if t is not None:
            t.record_stream(stream)


def winner_buffer(d: dict, device) -> torch.Tensor:
    return torch.empty(tconv_winner_bytes(d), dtype=torch.uint8, device=device)


def forward(d: dict, x, w, w2=None, alpha=None, beta=None, bias=None, want_winners=False,
            stream=None):
    """Allocate y (and the winner buffer) and run tconv_forward.  Returns (y, winners)."""
    N, C, H, W, K, R, S = (d[k] for k in "NCHWKRS")
    dt = TORCH_DTYPE[d["dtype"]]
    _check(x, (N, C, H, W), _x_dtype(d), "x"); _check(w, (K, C, R, S), dt, "w"); _check(w2, (K, C, R, S), dt, "w2")
    _check(alpha, (K, C), torch.float32, "alpha"); _check(beta, (K, C), torch.float32, "beta")
    _check(bias, (K,), torch.float32, "bias")
    OH, OW = tconv_output_shape(d)
    y = torch.empty((N, K, OH, OW), dtype=dt, device=x.device)
    winners = winner_buffer(d, x.device) if want_winners else None
    nws = tconv_workspace_bytes(d, False)
    ws = torch.empty(nws, dtype=torch.uint8, device=x.device) if nws else None
    _on_stream(stream, y, winners, ws)
    rc = tconv_forward(d, x, w, w2, alpha, beta, bias, y, winners, ws, stream)
    if rc != 0:
        raise TconvError(rc, "tconv_forward")
    return y, winners


def forward_stats(d: dict, x, w, w2=None, alpha=None, beta=None, bias=None, want_winners=False, stream=None):
    """forward() that also returns the per-channel sums of y and of y^2 (fp32 [K] each), taken in
    the kernel's epilogue.  Returns (y, winners, sum_y, sum_y2)."""
    N, C, H, W, K, R, S = (d[k] for k in "NCHWKRS")
    dt = TORCH_DTYPE[d["dtype"]]
    _check(x, (N, C, H, W), _x_dtype(d), "x"); _check(w, (K, C, R, S), dt, "w"); _check(w2, (K, C, R, S), dt, "w2")
    _check(alpha, (K, C), torch.float32, "alpha"); _check(beta, (K, C), torch.float32, "beta")
    _check(bias, (K,), torch.float32, "bias")
    OH, OW = tconv_output_shape(d)
    y = torch.empty((N, K, OH, OW), dtype=dt, device=x.device)
    winners = winner_buffer(d, x.device) if want_winners else None
    sum_y = torch.empty((K,), dtype=torch.float32, device=x.device)
    sum_y2 = torch.empty((K,), dtype=torch.float32, device=x.device)
    ws = torch.empty(tconv_stats_workspace_bytes(d), dtype=torch.uint8, device=x.device)
    _on_stream(stream, y, winners, sum_y, sum_y2, ws)
    rc = tconv_forward_stats(d, x, w, w2, alpha, beta, bias, y, winners, sum_y, sum_y2, ws, stream)
    if rc != 0:
        raise TconvError(rc, "tconv_forward_stats")
    return y, winners, sum_y, sum_y2


def backward(d: dict, x, w, grad_y, w2=None, alpha=None, beta=None, winners=None, stream=None,
             need=("grad_x", "grad_w", "grad_w2", "grad_alpha", "grad_beta", "grad_bias")):
    """Allocate the gradients named in `need` and run tconv_backward.  Returns a dict."""
    N, C, H, W, K, R, S = (d[k] for k in "NCHWKRS")
    dt = TORCH_DTYPE[d["dtype"]]
    OH, OW = tconv_output_shape(d)
    _check(x, (N, C, H, W), _x_dtype(d), "x"); _check(w, (K, C, R, S), dt, "w"); _check(w2, (K, C, R, S), dt, "w2")
    _check(grad_y, (N, K, OH, OW), dt, "grad_y")
    two = d["mode"] in ("compound", "parallel")
    dev = x.device
    f32 = torch.float32
    out = {}
    if "grad_x" in need:
        out["grad_x"] = torch.empty((N, C, H, W), dtype=dt, device=dev)
    if "grad_w" in need:
        out["grad_w"] = torch.empty((K, C, R, S), dtype=f32, device=dev)
    if "grad_w2" in need and d["mode"] == "parallel":
        out["grad_w2"] = torch.empty((K, C, R, S), dtype=f32, device=dev)
    if "grad_alpha" in need and two:
        out["grad_alpha"] = torch.empty((K, C), dtype=f32, device=dev)
    if "grad_beta" in need and two:
        out["grad_beta"] = torch.empty((K, C), dtype=f32, device=dev)
    if "grad_bias" in need:
        out["grad_bias"] = torch.empty((K,), dtype=f32, device=dev)
    nws = tconv_workspace_bytes(d, True)
    if winners is not None:
        # the figure includes room for recomputed winners, not needed when they are passed
        nws -= (tconv_winner_bytes(d) + 255) // 256 * 256
    ws = torch.empty(nws, dtype=torch.uint8, device=dev) if nws > 0 else None
    _on_stream(stream, ws, *out.values())
    rc = tconv_backward(d, x, w, w2, alpha, beta, grad_y, winners, out.get("grad_x"),
                        out.get("grad_w"), out.get("grad_w2"), out.get("grad_alpha"),
                        out.get("grad_beta"), out.get("grad_bias"), ws, stream)
    if rc != 0:
        raise TconvError(rc, "tconv_backward")
    return out


def dw_forward(d: dict, x, w, w2=None, alpha=None, beta=None, bias=None, want_winners=False, stream=None):
    """Depthwise form: allocate y (and the winner codes) and run tconv_dw_forward.  Returns (y, winners)."""
    N, C, H, W, R, S = (d[k] for k in "NCHWRS")
    dt = TORCH_DTYPE[d["dtype"]]
    _check(x, (N, C, H, W), dt, "x"); _check(w, (C, R, S), dt, "w"); _check(w2, (C, R, S), dt, "w2")
    _check(alpha, (C,), torch.float32, "alpha"); _check(beta, (C,), torch.float32, "beta")
    _check(bias, (C,), torch.float32, "bias")
    OH, OW = tconv_output_shape(d)
    y = torch.empty((N, C, OH, OW), dtype=dt, device=x.device)
    winners = torch.empty((N, C, OH, OW), dtype=torch.uint8, device=x.device) if want_winners else None
    _on_stream(stream, y, winners)
    rc = tconv_dw_forward(d, x, w, w2, alpha, beta, bias, y, winners, stream)
    if rc != 0:
        raise TconvError(rc, "tconv_dw_forward")
    return y, winners


def dw_backward(d: dict, x, w, grad_y, w2=None, alpha=None, beta=None, winners=None, stream=None):
    """Depthwise form: allocate every gradient the mode has and run tconv_dw_backward.  Returns a dict."""
    N, C, H, W, R, S = (d[k] for k in "NCHWRS")
    dt = TORCH_DTYPE[d["dtype"]]
    OH, OW = tconv_output_shape(d)
    _check(x, (N, C, H, W), dt, "x"); _check(w, (C, R, S), dt, "w"); _check(w2, (C, R, S), dt, "w2")
    _check(grad_y, (N, C, OH, OW), dt, "grad_y")
    two, par = d["mode"] in ("compound", "parallel"), d["mode"] == "parallel"
    dev, f32 = x.device, torch.float32
    out = {"grad_x": torch.empty((N, C, H, W), dtype=dt, device=dev),
           "grad_w": torch.empty((C, R, S), dtype=f32, device=dev),
           "grad_bias": torch.empty((C,), dtype=f32, device=dev)}
    if par:
        out["grad_w2"] = torch.empty((C, R, S), dtype=f32, device=dev)
    if two:
        out["grad_alpha"] = torch.empty((C,), dtype=f32, device=dev)
        out["grad_beta"] = torch.empty((C,), dtype=f32, device=dev)
    ws = torch.empty(tconv_dw_workspace_bytes(d, True), dtype=torch.uint8, device=dev)
    _on_stream(stream, ws, *out.values())
    rc = tconv_dw_backward(d, x, w, w2, alpha, beta, grad_y, winners, out["grad_x"], out["grad_w"],
                           out.get("grad_w2"), out.get("grad_alpha"), out.get("grad_beta"),
                           out["grad_bias"], ws, stream)
    if rc != 0:
        raise TconvError(rc, "tconv_dw_backward")
    return out
