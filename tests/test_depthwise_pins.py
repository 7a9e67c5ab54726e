"""Pins of the depthwise (groups = C) oracle wrappers against things other than the oracle:
a numpy unfold / min / max formulation written out per channel, torch's max_pool2d for the
zero-weight max-plus layer, the depthwise specialisation of conv2d for 1x1 windows, and gradient
conservation."""
import numpy as np
import pytest
import torch

from oracle import tconv_oracle as ora
import unfold_ref


def _draw(d, seed, par=False):
    rs = np.random.RandomState(seed)
    N, C, H, W, R, S = d["N"], d["C"], d["H"], d["W"], d["R"], d["S"]
    OH, OW = ora.output_shape(d)
    t = dict(x=rs.standard_normal((N, C, H, W)).astype(np.float32),
             w=(0.3 * rs.standard_normal((C, R, S))).astype(np.float32),
             w2=(0.3 * rs.standard_normal((C, R, S))).astype(np.float32),
             alpha=rs.uniform(-1, 1, C).astype(np.float32), beta=rs.uniform(-1, 1, C).astype(np.float32),
             bias=rs.uniform(-0.1, 0.1, C).astype(np.float32),
             g=rs.standard_normal((N, C, OH, OW)).astype(np.float32))
    return t


@pytest.mark.parametrize("mode", ["max_plus", "min_plus", "compound", "parallel"])
@pytest.mark.parametrize("geom", [dict(stride=(1, 1), pad=(1, 1), dil=(1, 1)), dict(stride=(2, 2), pad=(1, 1), dil=(1, 1)),
                                  dict(stride=(1, 2), pad=(2, 0), dil=(2, 1))])
def test_depthwise_is_the_per_channel_window_extremum(mode, geom):
    d = ora.make_desc(2, 5, 9, 11, 5, 3, 3, mode=mode, **geom)
    t = _draw(d, 31)
    two, par = mode in ("compound", "parallel"), mode == "parallel"
    got = ora.depthwise_forward(d, t["x"], t["w"], t["w2"] if par else None,
                                t["alpha"] if two else None, t["beta"] if two else None, t["bias"])
    p = unfold_ref.unfold(d, t["x"])                                  # [N,C,RS,OH,OW]
    ta = p + t["w"].reshape(1, 5, 9, 1, 1)
    tb = p + t["w2"].reshape(1, 5, 9, 1, 1) if par else ta
    mn, mx = ta.min(2), tb.max(2)
    if two:
        a, b = t["alpha"].reshape(1, 5, 1, 1), t["beta"].reshape(1, 5, 1, 1)
        y = unfold_ref.fmaf32(b, mx, unfold_ref.fmaf32(a, mn, np.zeros_like(mn)))
        codes = (ta.argmin(2) | (tb.argmax(2) << 4)).astype(np.uint8)
    elif mode == "max_plus":
        y, codes = mx, (tb.argmax(2) << 4).astype(np.uint8)
    else:
        y, codes = mn, ta.argmin(2).astype(np.uint8)
    y = (y + t["bias"].reshape(1, 5, 1, 1)).astype(np.float32)
    assert np.array_equal(got["y"].view(np.uint32), y.view(np.uint32))
    assert np.array_equal(got["codes"], codes)


def test_zero_weight_max_plus_depthwise_is_max_pooling():
    d = ora.make_desc(2, 4, 10, 12, 4, 3, 3, stride=(2, 2), pad=(1, 1), mode="max_plus")
    t = _draw(d, 32)
    x = np.abs(t["x"])      # non-negative input: zero padding equals max_pool2d's -inf padding
    got = ora.depthwise_forward(d, x, np.zeros((4, 3, 3), np.float32))
    ref = torch.nn.functional.max_pool2d(torch.from_numpy(x), 3, stride=2, padding=1).numpy()
    assert np.array_equal(got["y"], ref)


def test_one_by_one_compound_depthwise_is_a_depthwise_conv2d():
    """1x1 window: min = max = x + w, so y = (alpha + beta) * (x + w) + bias."""
    d = ora.make_desc(2, 6, 5, 7, 6, 1, 1, mode="compound")
    t = _draw(d, 33)
    got = ora.depthwise_forward(d, t["x"], t["w"], None, t["alpha"], t["beta"], t["bias"])
    s = (t["alpha"].astype(np.float64) + t["beta"].astype(np.float64))
    xw = t["x"].astype(np.float64) + t["w"].reshape(1, 6, 1, 1)
    ref = torch.nn.functional.conv2d(torch.from_numpy(xw), torch.from_numpy(s).reshape(6, 1, 1, 1),
                                     torch.from_numpy(t["bias"].astype(np.float64)), groups=6).numpy()
    assert np.allclose(got["y"], ref, rtol=1e-6, atol=1e-6)


@pytest.mark.parametrize("mode", ["max_plus", "compound", "parallel"])
def test_depthwise_gradients_conserve_the_upstream_gradient(mode):
    """Every output routes coef * g to exactly one tap per branch: per channel, grad_w sums to
    coef * sum(g), grad_bias to sum(g); grad_x sums to the same minus what fell into the padding."""
    d = ora.make_desc(3, 4, 8, 9, 4, 3, 3, pad=(0, 0), mode=mode)     # no padding: nothing is lost
    t = _draw(d, 34)
    two, par = mode in ("compound", "parallel"), mode == "parallel"
    gr = ora.depthwise_backward(d, t["x"], t["w"], t["g"], t["w2"] if par else None,
                                t["alpha"] if two else None, t["beta"] if two else None)
    sg = t["g"].astype(np.float64).sum((0, 2, 3))
    a = t["alpha"].astype(np.float64) if two else np.ones(4)
    b = t["beta"].astype(np.float64) if two else np.zeros(4)
    if mode == "max_plus":
        a, b = np.zeros(4), np.ones(4)
    assert np.allclose(gr["grad_bias"][0], sg)
    if par:
        assert np.allclose(gr["grad_w"][0].sum((1, 2)), a * sg) and np.allclose(gr["grad_w2"][0].sum((1, 2)), b * sg)
    else:
        assert np.allclose(gr["grad_w"][0].sum((1, 2)), (a + b) * sg)
    assert np.allclose(gr["grad_x"][0].sum((0, 2, 3)), (a + b) * sg)
