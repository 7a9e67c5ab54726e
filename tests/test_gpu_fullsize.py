"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

The oracle cannot run a whole full-size layer in seconds, so it computes a sample one piece
at a time: a few images x a slice of output channels.  The forward outputs and winners of
that sample are compared bit for bit with the full-size GPU run.  For the backward pass the
upstream gradient is zeroed outside the sample; then grad_x of the sampled images and the
parameter gradients of the sampled output channels equal what the oracle computes on the
sliced problem, and every other gradient element must be exactly zero.
"""
import numpy as np
import pytest
import torch

from oracle import tconv_oracle as ora
from paper_2504_06881_b200 import inputs, tconv
import parity

pytestmark = pytest.mark.gpu


def full_size_check(d, dist, seed, sample_n, sample_k):
    t = inputs.draw(d, seed, **dist)
    dt = tconv.TORCH_DTYPE[d["dtype"]]
    two = d["mode"] in ("compound", "parallel")
    par = d["mode"] == "parallel"
    k0, k1 = sample_k
    # upstream gradient: zero outside the sample
    gm = np.zeros_like(t["g"])
    for n in sample_n:
        gm[n, k0:k1] = t["g"][n, k0:k1]
    dev = {k: torch.from_numpy(v).cuda() for k, v in t.items()}
    for k in ("x", "w", "w2"):
        dev[k] = dev[k].to(dt)
    gdev = torch.from_numpy(gm).cuda().to(dt)
    y, win = tconv.forward(d, dev["x"], dev["w"], dev["w2"] if par else None,
                           dev["alpha"] if two else None, dev["beta"] if two else None, dev["bias"],
                           want_winners=True)
    kernel_fwd = tconv.tconv_last_kernel()
    grads = tconv.backward(d, dev["x"], dev["w"], gdev, dev["w2"] if par else None,
                           dev["alpha"] if two else None, dev["beta"] if two else None, win)
    torch.cuda.synchronize()
    assert tconv.tconv_device_status() == 0
    assert "tiled" in kernel_fwd, kernel_fwd
    wn = parity.winners_as_numpy(d, win)
    ds = dict(d, N=1, K=k1 - k0)
    sl = lambda a: np.ascontiguousarray(a[k0:k1])
    al, be = (sl(t["alpha"]), sl(t["beta"])) if two else (None, None)
    acc = {}
    for n in sample_n:
        xs = np.ascontiguousarray(t["x"][n:n + 1])
        ref = ora.forward(ds, xs, sl(t["w"]), sl(t["w2"]) if par else None, al, be, sl(t["bias"]))
        yg = y[n, k0:k1].float().cpu().numpy()
        assert parity.same_bits(yg, ref["y"][0]).all(), (d["mode"], n, "forward differs")
        want = ref["idx"] if ref["idx"] is not None else ref["codes"]
        assert np.array_equal(wn[n, k0:k1], want[0]), (d["mode"], n, "winners differ")
        rb = ora.backward(ds, xs, sl(t["w"]), np.ascontiguousarray(gm[n:n + 1, k0:k1]),
                          sl(t["w2"]) if par else None, al, be)
        parity.compare_grads(d, {"grad_x": grads["grad_x"][n:n + 1]}, {"grad_x": rb["grad_x"]})
        for name, (gv, ga) in rb.items():
            if name == "grad_x":
                continue
            if name not in acc:
                acc[name] = [np.zeros_like(gv), np.zeros_like(ga)]
            acc[name][0] += gv
            acc[name][1] += ga
    # parameter gradients of the sampled channels, zeros elsewhere
    for name, (gv, ga) in acc.items():
        got = grads[name]
        parity.compare_grads(d, {name: got[k0:k1]}, {name: (gv, ga)})
        rest = torch.cat([got[:k0], got[k1:]])
        assert torch.count_nonzero(rest) == 0, name
    others = [n for n in range(d["N"]) if n not in sample_n]
    assert torch.count_nonzero(grads["grad_x"][others[:4]]) == 0
    return kernel_fwd


@pytest.mark.parametrize("mode", ["max_plus", "min_plus", "compound", "parallel"])
def test_cfg2_full_size(mode):
    """N=128, C=K=64, 32x32, fp32: the step bench.py times."""
    d, dist = inputs.cfg2(mode)
    k = full_size_check(d, dist, 1020, sample_n=(0, 77, 127), sample_k=(24, 40))
    assert "tma" in k


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_cfg3a_full_size(dtype):
    """ImageNet-scale mid layer, parallel, N=64, C=K=128, 28x28."""
    d, dist = inputs.cfg3a(dtype)
    full_size_check(d, dist, 1030, sample_n=(5, 63), sample_k=(120, 128))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_cfg3b_full_size(dtype):
    """Stride-2 variant, C=64 -> K=128 from 56x56."""
    d, dist = inputs.cfg3b(dtype)
    full_size_check(d, dist, 1031, sample_n=(0, 31), sample_k=(0, 8))


def test_cfg4_full_size():
    """Segmentation-scale map, compound bf16, N=8, C=K=256, 128x256, dilation 2."""
    d, dist = inputs.cfg4("bf16")
    k = full_size_check(d, dist, 1040, sample_n=(7,), sample_k=(100, 102))
    assert "bf16_tma" in k
