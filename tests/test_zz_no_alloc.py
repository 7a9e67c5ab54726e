"""The allocation-free forward entry point (collected last on purpose: if it fails, a run that
stops at the first failure has already run every other test).

tconv_forward_noalloc serves callers that cannot hand the library a workspace because they
must not allocate device memory (a fixed-budget real-time loop, a plug-in whose host owns
all device memory, a plain C program without an allocator of its own).  It must give exactly what tconv_forward
gives, call after call, although every call reuses the same built-in scratch."""
import numpy as np
import pytest
import torch

from oracle import tconv_oracle as ora
from paper_2504_06881_b200 import inputs, tconv
import parity


def _layers():
    return [inputs.layer(3, 19, 20, 32, 41, 3, 3, stride=1, pad=1, mode="parallel"),       # TMA-staged
            inputs.layer(2, 10, 30, 29, 35, 3, 3, stride=2, pad=1, mode="compound"),       # per-element staging
            inputs.layer(2, 7, 16, 16, 9, 3, 3, stride=1, pad=1, mode="max_plus"),
            inputs.layer(2, 12, 24, 32, 20, 3, 3, stride=1, pad=1, mode="compound", dtype="bf16"),
            inputs.layer(2, 6, 14, 16, 8, 5, 5, stride=1, pad=2, mode="min_plus", chan="sum")]   # 16-bit codes


def _args(d, dev):
    two = d["mode"] in ("compound", "parallel")
    return (dev["x"], dev["w"], dev["w2"] if d["mode"] == "parallel" else None,
            dev["alpha"] if two else None, dev["beta"] if two else None, dev["bias"])


@pytest.mark.gpu
def test_noalloc_forward_matches_forward_on_two_calls_in_a_row():
    assert tconv.tconv_forward_noalloc_max_scratch() == 8 << 20
    layers = _layers()
    for i, d in enumerate(layers):
        t = inputs.draw(d, 900 + i)
        dev = parity.to_dev(t, d)
        want, want_win = tconv.forward(d, *_args(d, dev), want_winners=True)
        kernel = tconv.tconv_last_kernel()
        # the output the existing entry point gives is the oracle's (bit for bit)
        la = parity.layer_args(d, t)
        ref = ora.forward(d, t["x"], t["w"], la["w2"], la["alpha"], la["beta"], t["bias"])
        assert parity.same_bits(want.float().cpu().numpy(), ref["y"]).all(), d
        # a second layer in between, so that the shared scratch holds another layer's data
        other = layers[(i + 1) % len(layers)]
        to = parity.to_dev(inputs.draw(other, 950 + i), other)
        yo = torch.empty((other["N"], other["K"]) + tconv.tconv_output_shape(other), device="cuda",
                         dtype=tconv.TORCH_DTYPE[other["dtype"]])
        y = torch.empty_like(want)
        win = torch.empty_like(want_win)
        torch.cuda.synchronize()
        held = torch.cuda.memory_allocated()
        for call in range(2):
            y.fill_(float("nan"))
            win.zero_()
            rc = tconv.tconv_forward_noalloc(d, *_args(d, dev), y, win)
            assert rc == 0, tconv.tconv_status_string(rc)
            assert tconv.tconv_last_kernel() == kernel
            torch.cuda.synchronize()
            # the tolerance of the forward parity tests: bit-exact, against the existing entry
            # point and against the oracle
            assert torch.equal(y, want), (d, call)
            assert torch.equal(win, want_win), (d, call)
            assert parity.same_bits(y.float().cpu().numpy(), ref["y"]).all(), (d, call)
            rc = tconv.tconv_forward_noalloc(other, *_args(other, to), yo, None)
            assert rc == 0
        torch.cuda.synchronize()
        # nothing was allocated through the framework's allocator by the calls themselves
        assert torch.cuda.memory_allocated() == held
        assert tconv.tconv_device_status() == 0


def test_noalloc_forward_rejects_layers_beyond_its_scratch():
    """Host-side check, no GPU needed: a layer whose scratch exceeds the built-in array is
    refused before anything is launched."""
    import ctypes
    d = inputs.layer(1, 1024, 8, 8, 1024, 3, 3, pad=1, mode="parallel")
    assert tconv.tconv_workspace_bytes(d, False) > tconv.tconv_forward_noalloc_max_scratch()
    lib = ctypes.CDLL(str(tconv.LIB_PATH))
    lib.tconv_forward_noalloc.restype = ctypes.c_int
    vp = ctypes.c_void_p
    desc = tconv.make_desc(d)
    args = [ctypes.byref(desc), vp(0x1000), vp(0x1000), vp(0x1000), vp(0), vp(0), vp(0), vp(0x1000), vp(0), vp(0)]
    assert lib.tconv_forward_noalloc(*args) == -7
    assert b"scratch" in ctypes.cast(lib.tconv_last_error, ctypes.CFUNCTYPE(ctypes.c_char_p))()
