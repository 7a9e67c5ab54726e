"""The allocation-free forward entry point (collected last on purpose: if it fails, a run that
stops at the first failure has already run every other test).

tconv_forward_noalloc serves callers that cannot hand the library a workspace because they
must not allocate device memory (inside a stream capture, in a fixed-budget real-time loop,
in a plug-in whose host owns all device memory).  It must give exactly what tconv_forward
gives, call after call, although every call reuses the same built-in scratch."""
import pytest
import torch

from paper_2504_06881_b200 import inputs, tconv


def _layers():
    return [inputs.layer(3, 19, 20, 32, 41, 3, 3, stride=1, pad=1, mode="parallel"),       # TMA-staged
            inputs.layer(2, 10, 30, 29, 35, 3, 3, stride=2, pad=1, mode="compound"),       # per-element staging
            inputs.layer(2, 7, 16, 16, 9, 3, 3, stride=1, pad=1, mode="max_plus")]


@pytest.mark.gpu
def test_noalloc_forward_matches_forward_on_two_calls_in_a_row():
    assert tconv.tconv_forward_noalloc_max_scratch() == 8 << 20
    for i, d in enumerate(_layers()):
        t = inputs.draw(d, 900 + i)
        dev = {k: torch.from_numpy(v).cuda() for k, v in t.items()}
        two = d["mode"] in ("compound", "parallel")
        w2 = dev["w2"] if d["mode"] == "parallel" else None
        al, be = (dev["alpha"], dev["beta"]) if two else (None, None)
        want, want_win = tconv.forward(d, dev["x"], dev["w"], w2, al, be, dev["bias"], want_winners=True)
        kernel = tconv.tconv_last_kernel()
        # second layer in between, so that the shared scratch holds another layer's data
        other = _layers()[(i + 1) % 3]
        to = {k: torch.from_numpy(v).cuda() for k, v in inputs.draw(other, 950 + i).items()}
        for call in range(2):
            y = torch.full_like(want, float("nan"))
            win = torch.zeros_like(want_win)
            rc = tconv.tconv_forward_noalloc(d, dev["x"], dev["w"], w2, al, be, dev["bias"], y, win)
            assert rc == 0, tconv.tconv_status_string(rc)
            assert tconv.tconv_last_kernel() == kernel
            torch.cuda.synchronize()
            # the tolerance of the forward parity tests: bit-exact
            assert torch.equal(y, want), (d, call)
            assert torch.equal(win, want_win), (d, call)
            otwo = other["mode"] in ("compound", "parallel")
            yo = torch.empty((other["N"], other["K"]) + tconv.tconv_output_shape(other), device="cuda")
            rc = tconv.tconv_forward_noalloc(other, to["x"], to["w"],
                                             to["w2"] if other["mode"] == "parallel" else None,
                                             to["alpha"] if otwo else None, to["beta"] if otwo else None,
                                             to["bias"], yo, None)
            assert rc == 0
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
