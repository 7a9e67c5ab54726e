"""Parity of the three-dimensional kernels with the three-dimensional oracle: forward outputs and
winners bit for bit, gradients within the tolerance of the dense layers (1e-5 fp32, 2e-2 bf16 of
the sum of |contributions|).  Shapes cover the paper's 3-D LeNet layers (5 x 5 x 5 windows, one
to sixteen channels, stride 2 in the first layer), ragged volumes, strides, dilations and ties."""
import numpy as np
import pytest
import torch

from oracle import tconv3d_oracle as ora3
from paper_2504_06881_b200 import inputs, tconv, tconv3d
import parity

pytestmark = pytest.mark.gpu

MODES = [("max_plus", "default"), ("min_plus", "default"), ("max_plus", "sum"), ("min_plus", "sum"),
         ("max_plus", "min"), ("min_plus", "max"), ("compound", "default"), ("parallel", "default")]


def check(d, seed, dists=None, null_ab=False, use_bias=True):
    t = inputs.draw3d(d, seed, **(dists or {}))
    two, par = d["mode"] in ("compound", "parallel"), d["mode"] == "parallel"
    dt = tconv.TORCH_DTYPE[d["dtype"]]
    dev = lambda a, ty=None: torch.from_numpy(a).cuda().to(ty) if ty else torch.from_numpy(a).cuda()
    al = t["alpha"] if (two and not null_ab) else None
    be = t["beta"] if (two and not null_ab) else None
    bias = t["bias"] if use_bias else None
    ref = ora3.forward(d, t["x"], t["w"], t["w2"] if par else None, al, be, bias)
    gx, gw, gw2 = dev(t["x"], dt), dev(t["w"], dt), dev(t["w2"], dt) if par else None
    ga, gb = (dev(al) if al is not None else None), (dev(be) if be is not None else None)
    gbias = dev(bias) if use_bias else None
    y, win = tconv3d.forward(d, gx, gw, gw2, ga, gb, gbias, want_winners=True)
    y0, _ = tconv3d.forward(d, gx, gw, gw2, ga, gb, gbias, want_winners=False)
    torch.cuda.synchronize()
    want = inputs.to_bf16_values(ref["y"]) if d["dtype"] == "bf16" else ref["y"]
    for out in (y, y0):
        assert parity.same_bits(out.float().cpu().numpy(), want).all(), d
    if ref["idx"] is not None:
        assert np.array_equal(win.cpu().numpy(), ref["idx"]), d
    else:
        assert np.array_equal(win.cpu().numpy().view(np.uint16), ref["codes"]), d
    gref = ora3.backward(d, t["x"], t["w"], t["g"], t["w2"] if par else None, al, be)
    for winners in (win, None):       # stored winners, then recomputed into the workspace
        got = tconv3d.backward(d, gx, gw, dev(t["g"], dt), gw2, ga, gb, winners)
        torch.cuda.synchronize()
        assert set(got) == set(gref)
        parity.compare_grads(d, got, gref)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("mode,chan", MODES)
def test_small_ragged_volume(mode, chan, dtype):
    d = inputs.layer3d(2, 3, 7, 9, 11, 5, T=3, R=2, S=3, stride=(1, 2, 1), pad=(1, 0, 2), dil=(2, 1, 1),
                       mode=mode, chan=chan, dtype=dtype)
    check(d, 301)


@pytest.mark.parametrize("mode", ["max_plus", "compound", "parallel"])
@pytest.mark.parametrize("size,batch", [(28, 4), (64, 1)])
def test_lenet3d_first_layer(mode, size, batch):
    """[5/6, 2]: one input channel, six output channels, 5 x 5 x 5 window, stride 2."""
    d = inputs.layer3d(batch, 1, size, size, size, 6, T=5, R=5, S=5, stride=2, mode=mode)
    check(d, 302)


@pytest.mark.parametrize("mode", ["min_plus", "compound", "parallel"])
def test_lenet3d_second_layer(mode):
    """[5/16]: six to sixteen channels, 5 x 5 x 5 window, on the pooled 15^3 volume of the 64^3 net."""
    d = inputs.layer3d(2, 6, 15, 15, 15, 16, T=5, R=5, S=5, mode=mode)
    check(d, 303)


@pytest.mark.parametrize("mode,chan", MODES)
def test_integer_inputs_with_ties(mode, chan):
    d = inputs.layer3d(2, 4, 6, 6, 6, 3, T=3, R=3, S=3, pad=1, mode=mode, chan=chan)
    check(d, 304, dists=dict(x=("ints", -1, 1), w=("ints", -1, 1)))


def test_many_channels_span_several_weight_chunks():
    d = inputs.layer3d(1, 40, 6, 6, 8, 9, T=3, R=3, S=3, pad=1, mode="parallel")
    check(d, 305)
    check(dict(d, mode="max_plus", K=5), 306)


def test_parameter_free_and_no_bias():
    d = inputs.layer3d(2, 2, 5, 6, 7, 4, T=2, R=2, S=2, mode="compound")
    check(d, 307, null_ab=True, use_bias=False)


def test_largest_window_and_unit_window():
    check(inputs.layer3d(1, 2, 8, 8, 9, 2, T=4, R=8, S=8, pad=(1, 3, 3), mode="compound"), 308)
    check(inputs.layer3d(2, 3, 3, 4, 5, 2, T=1, R=1, S=1, mode="parallel"), 309)
