"""Pins of the CPU oracle against things other than itself (no GPU needed).

The paper prints no worked numeric example of a tropical convolution, so the
oracle is pinned by: a second formulation built from numpy library routines
(the paper's unfold -> add -> min/max -> channel-combine pipeline), library
special cases (max pooling, ordinary convolution), closed forms, the paper's
operation counts and parameter counts, algebraic invariants, hand-derived tie
cases, and exact piecewise-linearity of the forward map for the backward pass.
"""
import itertools
from pathlib import Path

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import tconv_oracle as ora
from paper_2504_06881_b200 import inputs
import unfold_ref

ALL_MODES = [("max_plus", "max"), ("min_plus", "min"), ("max_plus", "sum"), ("min_plus", "sum"),
             ("max_plus", "min"), ("min_plus", "max"), ("compound", "sum"), ("parallel", "sum")]
DYADIC = dict(x=("dyadic", 8, 4), w=("dyadic", 8, 4), ab=("dyadic", 1, 1), bias=("dyadic", 4, 1),
              g=("dyadic", 2, 2))


def same_bits(a, b):
    """bitwise equality except that +0 and -0 count as equal."""
    a = np.asarray(a, np.float32); b = np.asarray(b, np.float32)
    return bool(np.all((a.view(np.uint32) == b.view(np.uint32)) | ((a == 0) & (b == 0))))


def run_fwd(d, t, **kw):
    two = d["mode"] in ("compound", "parallel")
    return ora.forward(d, t["x"], t["w"], t["w2"] if d["mode"] == "parallel" else None,
                       kw.get("alpha", t["alpha"] if two else None),
                       kw.get("beta", t["beta"] if two else None),
                       kw.get("bias", t["bias"]))


# ---------------------------------------------------------------- P1
GEOMS = [(s, p, dl) for s in (1, 2) for p in (0, 1, 2) for dl in (1, 2)]


@pytest.mark.parametrize("mode,chan", ALL_MODES)
def test_p1_matches_unfold_formulation(mode, chan):
    """Whole forward and winners equal the numpy unfold/argmin/argmax formulation
    bit for bit, over every stride/pad/dilation in {1,2}x{0,1,2}x{1,2}."""
    for gi, (s, p, dl) in enumerate(GEOMS):
        for (H, W, R, S) in ((8, 7, 3, 3), (6, 8, 2, 3)):
            d = inputs.layer(2, 3, H, W, 4, R, S, stride=s, pad=p, dil=dl, mode=mode, chan=chan)
            if min(inputs.output_hw(d)) <= 0:
                continue
            t = inputs.draw(d, 100 + gi)
            o = run_fwd(d, t)
            two = mode in ("compound", "parallel")
            y, idx, codes = unfold_ref.forward(d, t["x"], t["w"], t["w2"],
                                               t["alpha"] if two else None,
                                               t["beta"] if two else None, t["bias"])
            assert same_bits(o["y"], y), (mode, chan, s, p, dl)
            if idx is not None:
                assert np.array_equal(o["idx"], idx)
            else:
                assert np.array_equal(o["codes"], codes)


def test_p1_asymmetric_geometry_and_5x5():
    """Different stride/pad/dilation per axis and a 5x5 window (the paper's LeNet kernel)."""
    d = inputs.layer(1, 2, 11, 9, 3, 5, 5, stride=(2, 1), pad=(2, 1), dil=(1, 1), mode="compound")
    t = inputs.draw(d, 7)
    o = ora.forward(d, t["x"], t["w"], None, None, None, t["bias"])
    y, _, codes = unfold_ref.forward(d, t["x"], t["w"], None, None, None, t["bias"])
    assert same_bits(o["y"], y)
    assert o["codes"] is None  # 25 taps do not fit a nibble
    d = inputs.layer(2, 2, 9, 10, 3, 3, 2, stride=(1, 2), pad=(0, 2), dil=(2, 1), mode="parallel")
    t = inputs.draw(d, 8)
    o = run_fwd(d, t)
    y, _, codes = unfold_ref.forward(d, t["x"], t["w"], t["w2"], t["alpha"], t["beta"], t["bias"])
    assert same_bits(o["y"], y) and np.array_equal(o["codes"], codes)


# ---------------------------------------------------------------- P2
@pytest.mark.parametrize("chan_max,chan_min", [("max", "min"), ("sum", "sum"), ("min", "max")])
def test_p2_min_max_duality(chan_max, chan_min):
    """min_plus(x, w) = -max_plus(-x, -w), with identical winners."""
    dmax = inputs.layer(2, 3, 7, 9, 4, 3, 3, stride=1, pad=1, mode="max_plus", chan=chan_max)
    dmin = dict(dmax, mode="min_plus", chan=chan_min)
    t = inputs.draw(dmax, 21)
    a = ora.forward(dmin, t["x"], t["w"], bias=t["bias"])
    b = ora.forward(dmax, -t["x"], -t["w"], bias=-t["bias"])
    assert same_bits(a["y"], -b["y"])
    if a["idx"] is not None:
        assert np.array_equal(a["idx"], b["idx"])
    else:
        assert np.array_equal(a["codes"], b["codes"] >> 4)


# ---------------------------------------------------------------- P3
@pytest.mark.parametrize("mode,chan", ALL_MODES)
def test_p3_weight_shift(mode, chan):
    """Adding delta to every weight moves y by delta (Max/Min combine), delta*C
    (Sum) or delta*sum_c(alpha+beta) (compound/parallel).  Dyadic-grid inputs
    make every fp32 operation exact, so the identity holds bit for bit."""
    d = inputs.layer(2, 4, 6, 7, 3, 3, 3, stride=1, pad=1, mode=mode, chan=chan)
    t = inputs.draw(d, 31, **DYADIC)
    delta = np.float32(0.75)
    y0 = run_fwd(d, t)["y"]
    t1 = dict(t, w=t["w"] + delta, w2=t["w2"] + delta)
    o1 = run_fwd(d, t1)
    if mode in ("compound", "parallel"):
        shift = delta * (t["alpha"] + t["beta"]).sum(axis=1)[None, :, None, None]
    elif chan == "sum":
        shift = delta * d["C"]
    else:
        shift = delta
    assert same_bits(o1["y"], y0 + np.float32(1) * shift)
    # the winners do not move
    o0 = run_fwd(d, t)
    key = "idx" if o0["idx"] is not None else "codes"
    assert np.array_equal(o0[key], o1[key])


# ---------------------------------------------------------------- P4
def test_p4_pointwise_single_channel_is_x_plus_w():
    """A 1x1 window with C_in = 1 leaves y = x + w (+ bias) in every mode."""
    for mode, chan in ALL_MODES:
        d = inputs.layer(2, 1, 5, 6, 3, 1, 1, mode=mode, chan=chan)
        t = inputs.draw(d, 41)
        half = np.full((3, 1), 0.5, np.float32)
        o = run_fwd(d, t, alpha=half if mode in ("compound", "parallel") else None,
                    beta=half if mode in ("compound", "parallel") else None)
        if mode == "parallel":
            # alpha*(x+w1) + beta*(x+w2) with alpha = beta = 0.5
            s1 = t["x"] + t["w"].reshape(1, 3, 1, 1)
            s2 = t["x"] + t["w2"].reshape(1, 3, 1, 1)
            want = unfold_ref.fmaf32(np.float32(0.5) * np.ones_like(s2), s2, np.float32(0.5) * s1)
            want = want + t["bias"].reshape(1, 3, 1, 1)
            assert np.allclose(o["y"], want, rtol=0, atol=1e-6)
            continue
        want = (t["x"] + t["w"].reshape(1, 3, 1, 1)) + t["bias"].reshape(1, 3, 1, 1)
        if mode == "compound":
            assert np.allclose(o["y"], want, rtol=0, atol=1e-6)  # 0.5*t + 0.5*t, one extra rounding
        else:
            assert same_bits(o["y"], want), (mode, chan)


# ---------------------------------------------------------------- P5
@pytest.mark.parametrize("stride,dil,R", [(1, 1, 3), (2, 1, 3), (1, 2, 3), (2, 2, 2), (3, 1, 2)])
def test_p5_zero_weight_is_max_pooling(stride, dil, R):
    """w = 0, no padding: MaxPlus-Max is max over channels of max_pool2d; MinPlus-Min via -x."""
    d = inputs.layer(2, 3, 11, 12, 2, R, R, stride=stride, pad=0, dil=dil, mode="max_plus")
    t = inputs.draw(d, 51)
    w0 = np.zeros_like(t["w"])
    y = ora.forward(d, t["x"], w0)["y"]
    pooled = F.max_pool2d(torch.from_numpy(t["x"]), R, stride=stride, dilation=dil).numpy()
    want = pooled.max(axis=1, keepdims=True).repeat(2, axis=1)
    assert same_bits(y, want)
    ymin = ora.forward(dict(d, mode="min_plus"), t["x"], w0)["y"]
    pooled = -F.max_pool2d(torch.from_numpy(-t["x"]), R, stride=stride, dilation=dil).numpy()
    assert same_bits(ymin, pooled.min(axis=1, keepdims=True).repeat(2, axis=1))
    # Sum combine: sum over channels of the pooled maps, channels ascending
    ysum = ora.forward(dict(d, chan="sum"), t["x"], w0)["y"]
    pooled = F.max_pool2d(torch.from_numpy(t["x"]), R, stride=stride, dilation=dil).numpy()
    acc = np.zeros_like(pooled[:, 0])
    for c in range(3):
        acc = acc + pooled[:, c]
    assert same_bits(ysum, acc[:, None].repeat(2, axis=1))


# ---------------------------------------------------------------- P6
def test_p6_zero_input_gives_constant_maps_including_borders():
    """x = 0 with zero padding: every output of channel k equals max_{c,r,s} w[k] + bias[k],
    at the border as in the interior (padded taps take part as x = 0)."""
    d = inputs.layer(1, 3, 6, 6, 4, 3, 3, stride=1, pad=2, dil=2, mode="max_plus")
    t = inputs.draw(d, 61)
    x0 = np.zeros_like(t["x"])
    y = ora.forward(d, x0, t["w"], bias=t["bias"])["y"]
    want = (t["w"].reshape(4, -1).max(axis=1) + t["bias"]).reshape(1, 4, 1, 1)
    assert same_bits(y, np.broadcast_to(want, y.shape))
    dc = dict(d, mode="compound")
    y = ora.forward(dc, x0, t["w"], None, t["alpha"], t["beta"], None)["y"]
    assert np.all(y == y[:, :, :1, :1])


# ---------------------------------------------------------------- P7
def test_p7_pointwise_sum_form_is_ordinary_convolution():
    """R = S = 1, Sum combine: y = conv2d(x, ones) + sum_c w[k, c] (+ bias)."""
    d = inputs.layer(2, 5, 6, 7, 4, 1, 1, stride=2, mode="max_plus", chan="sum")
    t = inputs.draw(d, 71)
    y = ora.forward(d, t["x"], t["w"], bias=t["bias"])["y"]
    conv = F.conv2d(torch.from_numpy(t["x"]).double(), torch.ones(4, 5, 1, 1).double(), stride=2)
    want = conv.numpy() + t["w"].astype(np.float64).sum(axis=(1, 2, 3)).reshape(1, 4, 1, 1) \
        + t["bias"].reshape(1, 4, 1, 1)
    assert np.allclose(y, want, rtol=1e-6, atol=1e-5)
    # compound with alpha, beta: an ordinary convolution with weight (alpha+beta)
    dc = dict(d, mode="compound", chan="default")
    y = ora.forward(dc, t["x"], t["w"], None, t["alpha"], t["beta"], t["bias"])["y"]
    ab = (t["alpha"] + t["beta"]).astype(np.float64)
    conv = F.conv2d(torch.from_numpy(t["x"]).double(), torch.from_numpy(ab).reshape(4, 5, 1, 1), stride=2)
    want = conv.numpy() + (ab * t["w"].reshape(4, 5)).sum(axis=1).reshape(1, 4, 1, 1) \
        + t["bias"].reshape(1, 4, 1, 1)
    assert np.allclose(y, want, rtol=1e-5, atol=1e-5)


# ---------------------------------------------------------------- P8
def test_p8_degenerate_cases():
    """(alpha, beta) = (1, 0) is MinPlus-Sum and (0, 1) is MaxPlus-Sum (remark after
    Definition 3); parallel with w1 = w2 is compound; missing alpha/beta mean ones."""
    d = inputs.layer(2, 3, 7, 6, 4, 3, 3, stride=1, pad=1, mode="compound")
    t = inputs.draw(d, 81)
    one, zero = np.ones((4, 3), np.float32), np.zeros((4, 3), np.float32)
    ymin = ora.forward(dict(d, mode="min_plus", chan="sum"), t["x"], t["w"], bias=t["bias"])["y"]
    ymax = ora.forward(dict(d, mode="max_plus", chan="sum"), t["x"], t["w"], bias=t["bias"])["y"]
    assert same_bits(ora.forward(d, t["x"], t["w"], None, one, zero, t["bias"])["y"], ymin)
    assert same_bits(ora.forward(d, t["x"], t["w"], None, zero, one, t["bias"])["y"], ymax)
    dp = dict(d, mode="parallel")
    yc = ora.forward(d, t["x"], t["w"], None, t["alpha"], t["beta"], t["bias"])
    yp = ora.forward(dp, t["x"], t["w"], t["w"].copy(), t["alpha"], t["beta"], t["bias"])
    assert same_bits(yc["y"], yp["y"]) and np.array_equal(yc["codes"], yp["codes"])
    y_null = ora.forward(d, t["x"], t["w"], None, None, None, t["bias"])["y"]
    assert same_bits(y_null, ora.forward(d, t["x"], t["w"], None, one, one, t["bias"])["y"])
    # parallel with (1,0) uses w1 only, with (0,1) w2 only
    y10 = ora.forward(dp, t["x"], t["w"], t["w2"], one, zero, t["bias"])["y"]
    y01 = ora.forward(dp, t["x"], t["w"], t["w2"], zero, one, t["bias"])["y"]
    assert same_bits(y10, ymin)
    assert same_bits(y01, ora.forward(dict(d, mode="max_plus", chan="sum"), t["x"], t["w2"],
                                      bias=t["bias"])["y"])


# ---------------------------------------------------------------- P9
@pytest.mark.parametrize("a,b", [(1.0, 1.0), (0.5, 0.5), (1.0, -1.0)])
def test_p9_compound_is_combination_of_separate_outputs(a, b):
    """Uniform alpha = a, beta = b (the fixed specialisations of the section
    "Specializations of compound/parallel tropical convolutions"):
    compound = a*MinPlusSum + b*MaxPlusSum, exactly on the dyadic grid."""
    d = inputs.layer(2, 4, 6, 6, 3, 3, 3, stride=1, pad=1, mode="compound")
    t = inputs.draw(d, 91, **DYADIC)
    A = np.full((3, 4), a, np.float32); B = np.full((3, 4), b, np.float32)
    yc = ora.forward(d, t["x"], t["w"], None, A, B, None)["y"]
    ymin = ora.forward(dict(d, mode="min_plus", chan="sum"), t["x"], t["w"])["y"]
    ymax = ora.forward(dict(d, mode="max_plus", chan="sum"), t["x"], t["w"])["y"]
    assert same_bits(yc, np.float32(a) * ymin + np.float32(b) * ymax)
    dp = dict(d, mode="parallel")
    yp = ora.forward(dp, t["x"], t["w"], t["w2"], A, B, None)["y"]
    ymax2 = ora.forward(dict(d, mode="max_plus", chan="sum"), t["x"], t["w2"])["y"]
    assert same_bits(yp, np.float32(a) * ymin + np.float32(b) * ymax2)


# ---------------------------------------------------------------- P10
@pytest.mark.parametrize("shape", [(1, 3, 7, 8, 4, 3, 3), (2, 5, 6, 6, 2, 2, 3), (1, 1, 5, 5, 3, 1, 1)])
def test_p10_operation_counts_match_section_4_1(shape):
    """Instrumented tallies equal the closed forms of the complexity analysis."""
    N, C, H, W, K, R, S = shape
    for mode, chan in ALL_MODES:
        d = inputs.layer(N, C, H, W, K, R, S, mode=mode, chan=chan)
        t = inputs.draw(d, 5)
        OH, OW = inputs.output_hw(d)
        P = N * K * OH * OW
        two = mode in ("compound", "parallel")
        cnt = ora.forward(d, t["x"], t["w"], t["w2"] if mode == "parallel" else None,
                          t["alpha"] if two else None, t["beta"] if two else None, None,
                          want_counts=True)["counts"]
        if mode == "compound":
            want = dict(muls=2 * C * P, adds=(R * S * C + 2 * C - 1) * P, cmps=2 * (R * S - 1) * C * P)
        elif mode == "parallel":
            want = dict(muls=2 * C * P, adds=(2 * R * S * C + 2 * C - 1) * P,
                        cmps=2 * (R * S - 1) * C * P)
        elif chan == "sum":
            want = dict(muls=0, adds=(C - 1 + R * S * C) * P, cmps=(R * S - 1) * C * P)
        else:
            want = dict(muls=0, adds=R * S * C * P, cmps=(R * S * C - 1) * P)
        assert cnt == want, (mode, chan, cnt, want)


# ---------------------------------------------------------------- P11
@pytest.mark.parametrize("mode,chan", ALL_MODES)
def test_p11_gradient_conservation(mode, chan):
    """Routing loses nothing: the window sums of grad_w reproduce grad_bias scaled by the
    branch coefficients, and with no padding grad_x sums to the same total.  Exact on the
    dyadic grid (float64 accumulation of dyadic numbers)."""
    d = inputs.layer(2, 3, 7, 7, 4, 3, 3, stride=1, pad=0, mode=mode, chan=chan)
    t = inputs.draw(d, 111, **DYADIC)
    two = mode in ("compound", "parallel")
    gr = ora.backward(d, t["x"], t["w"], t["g"], t["w2"] if mode == "parallel" else None,
                      t["alpha"] if two else None, t["beta"] if two else None)
    gbias = gr["grad_bias"][0]
    assert np.array_equal(gbias, t["g"].astype(np.float64).sum(axis=(0, 2, 3)))
    gw = gr["grad_w"][0]
    a = t["alpha"].astype(np.float64); b = t["beta"].astype(np.float64)
    if mode == "compound":
        assert np.array_equal(gw.sum(axis=(2, 3)), (a + b) * gbias[:, None])
        assert gr["grad_x"][0].sum() == ((a + b) * gbias[:, None]).sum()
    elif mode == "parallel":
        assert np.array_equal(gw.sum(axis=(2, 3)), a * gbias[:, None])
        assert np.array_equal(gr["grad_w2"][0].sum(axis=(2, 3)), b * gbias[:, None])
        assert gr["grad_x"][0].sum() == ((a + b) * gbias[:, None]).sum()
    elif chan == "sum":
        assert np.array_equal(gw.sum(axis=(2, 3)), np.broadcast_to(gbias[:, None], (4, 3)))
        assert gr["grad_x"][0].sum() == 3 * gbias.sum()
    else:
        assert np.array_equal(gw.sum(axis=(1, 2, 3)), gbias)
        assert gr["grad_x"][0].sum() == gbias.sum()
    # with padding, winners in the padding still feed grad_w but not grad_x
    dpad = dict(d, pad_h=2, pad_w=2)
    tp = inputs.draw(dpad, 112, **DYADIC)
    grp = ora.backward(dpad, tp["x"], tp["w"], tp["g"], tp["w2"] if mode == "parallel" else None,
                       tp["alpha"] if two else None, tp["beta"] if two else None)
    if not two and chan != "sum":
        assert np.array_equal(grp["grad_w"][0].sum(axis=(1, 2, 3)), grp["grad_bias"][0])
        assert abs(grp["grad_x"][1].sum()) <= np.abs(tp["g"]).sum()


# ---------------------------------------------------------------- P12
def _tie_free(d, seed):
    """Dyadic inputs whose taps never tie: grid 2^-4 plus a distinct 2^-10 offset per (c, tap)."""
    t = inputs.draw(d, seed, x=("dyadic", 4, 2), w=("dyadic", 4, 2), ab=("dyadic", 1, 1),
                    bias=("dyadic", 2, 1), g=("dyadic", 2, 2))
    C, RS = d["C"], d["R"] * d["S"]
    assert C * RS <= 64
    off = (np.arange(C * RS, dtype=np.float32) / 1024).reshape(1, C, d["R"], d["S"])
    t["w"] = t["w"] + off
    t["w2"] = t["w2"] + off[:, :, ::-1, ::-1]
    return t


@pytest.mark.parametrize("mode,chan", ALL_MODES)
@pytest.mark.parametrize("geom", [(1, 1, 1), (2, 1, 1), (1, 2, 2)])
def test_p12_backward_is_the_exact_directional_derivative(mode, chan, geom):
    """The forward map is piecewise linear.  For tie-free inputs and a perturbation too small
    to change any winner, L(x+eu, w+ev) - L(x, w) = e(<grad_x,u> + <grad_w,v>) with
    L = sum g*y.  All numbers sit on a dyadic grid, so both sides are exact."""
    s, p, dl = geom
    d = inputs.layer(2, 3, 7, 8, 3, 3, 3, stride=s, pad=p, dil=dl, mode=mode, chan=chan)
    t = _tie_free(d, 121)
    two = mode in ("compound", "parallel")
    par = mode == "parallel"
    rs = np.random.RandomState(5)
    eps = np.float32(2.0 ** -14)
    u = (rs.randint(-2, 3, t["x"].shape) / 2).astype(np.float32)
    v = (rs.randint(-2, 3, t["w"].shape) / 2).astype(np.float32)
    v2 = (rs.randint(-2, 3, t["w"].shape) / 2).astype(np.float32)
    al = t["alpha"] if two else None
    be = t["beta"] if two else None

    def L(x, w, w2, a, b):
        o = ora.forward(d, x, w, w2 if par else None, a, b, t["bias"])
        return (o["y"].astype(np.float64) * t["g"].astype(np.float64)).sum(), o

    L0, o0 = L(t["x"], t["w"], t["w2"], al, be)
    L1, o1 = L(t["x"] + eps * u, t["w"] + eps * v, t["w2"] + eps * v2, al, be)
    key = "idx" if o0["idx"] is not None else "codes"
    assert np.array_equal(o0[key], o1[key]), "perturbation moved a winner"
    gr = ora.backward(d, t["x"], t["w"], t["g"], t["w2"] if par else None, al, be)
    lin = (gr["grad_x"][0] * u).sum() + (gr["grad_w"][0] * v).sum()
    if par:
        lin += (gr["grad_w2"][0] * v2).sum()
    assert L1 - L0 == float(eps) * lin
    assert lin != 0
    if two:
        da = (rs.randint(-2, 3, al.shape) / 2).astype(np.float32)
        db = (rs.randint(-2, 3, al.shape) / 2).astype(np.float32)
        L2, _ = L(t["x"], t["w"], t["w2"], al + da, be + db)
        assert L2 - L0 == (gr["grad_alpha"][0] * da).sum() + (gr["grad_beta"][0] * db).sum()


def test_p12_abs_sums_bound_the_gradients():
    d = inputs.layer(2, 3, 6, 6, 4, 3, 3, pad=1, mode="parallel")
    t = inputs.draw(d, 122)
    gr = ora.backward(d, t["x"], t["w"], t["g"], t["w2"], t["alpha"], t["beta"])
    for name, (gv, ga) in gr.items():
        assert np.all(np.abs(gv) <= ga * (1 + 1e-12) + 1e-300), name


# ---------------------------------------------------------------- P13
def test_p13_ties_go_to_the_lowest_flattened_index_hand_case():
    """x = 0, w = 0: every tap ties; the winner is (c, r, s) = (0, 0, 0).  grad_w lands on
    that tap only; grad_x receives g shifted by the tap's offset (-pad), minus the padding."""
    d = inputs.layer(1, 2, 4, 4, 2, 3, 3, stride=1, pad=1, mode="max_plus")
    x = np.zeros((1, 2, 4, 4), np.float32); w = np.zeros((2, 2, 3, 3), np.float32)
    g = np.arange(32, dtype=np.float32).reshape(1, 2, 4, 4) + 1
    o = ora.forward(d, x, w)
    assert np.all(o["idx"] == 0) and np.all(o["y"] == 0)
    gr = ora.backward(d, x, w, g)
    gw = gr["grad_w"][0]
    assert gw[0, 0, 0, 0] == g[0, 0].sum() and gw[1, 0, 0, 0] == g[0, 1].sum()
    assert np.count_nonzero(gw) == 2
    gx = gr["grad_x"][0]
    want = np.zeros((1, 2, 4, 4))
    # output (oh, ow) reads input (oh-1, ow-1) at tap (0, 0)
    want[0, 0, :3, :3] = (g[0, 0] + g[0, 1])[1:, 1:]
    assert np.array_equal(gx, want)
    # Sum form: the winner is tap 0 in every channel, for both branches of compound
    dc = dict(d, mode="compound", chan="default")
    oc = ora.forward(dc, x, w)
    assert np.all(oc["codes"] == 0)
    grc = ora.backward(dc, x, w, g)
    assert np.count_nonzero(grc["grad_w"][0]) == 4
    assert grc["grad_w"][0][0, 1, 0, 0] == 2 * g[0, 0].sum()


def test_p13_integer_inputs_with_many_ties():
    """Small-integer inputs tie constantly; winners must equal numpy's first-occurrence
    argmin/argmax in every mode, and a one-tap bump must move the winner to that tap."""
    for mode, chan in ALL_MODES:
        d = inputs.layer(2, 3, 6, 7, 3, 3, 3, stride=1, pad=1, mode=mode, chan=chan)
        t = inputs.draw(d, 131, x=("ints", -1, 1), w=("ints", -1, 1))
        two = mode in ("compound", "parallel")
        o = run_fwd(d, t)
        y, idx, codes = unfold_ref.forward(d, t["x"], t["w"], t["w2"], t["alpha"] if two else None,
                                           t["beta"] if two else None, t["bias"])
        assert same_bits(o["y"], y)
        assert np.array_equal(o["idx"], idx) if idx is not None else np.array_equal(o["codes"], codes)
    d = inputs.layer(1, 2, 3, 3, 1, 3, 3, stride=1, pad=1, mode="max_plus")
    x = np.zeros((1, 2, 3, 3), np.float32)
    w = np.zeros((1, 2, 3, 3), np.float32)
    w[0, 1, 2, 1] = 1.0   # unique maximum at c=1, r=2, s=1 -> flattened 9 + 7
    assert np.all(ora.forward(d, x, w)["idx"] == 16)
    w[0, 0, 1, 2] = 1.0   # an equal value at a lower flattened index (5) now wins
    assert np.all(ora.forward(d, x, w)["idx"] == 5)


# ---------------------------------------------------------------- P14
def test_p14_parameter_counts_of_the_papers_lenets():
    """alpha/beta have one entry per (c_in, c_out), parallel adds one weight tensor and no
    second bias: the tensor shapes of this interface reproduce the paper's parameter counts."""
    golden = {}
    for line in (Path(__file__).parent / "golden" / "lenet_param_counts.txt").read_text().splitlines():
        if line and not line.startswith("#"):
            name, n = line.split()
            golden[name] = int(n)

    def layer_params(cin, cout, kind, nparam):
        d = inputs.layer(1, cin, 12, 12, cout, 5, 5, mode="parallel" if kind == "P" else "compound")
        t = inputs.draw(d, 0)
        n = t["w"].size + t["bias"].size
        if kind == "P":
            n += t["w2"].size
        if kind in ("C", "P"):
            n += nparam * t["alpha"].size
        return n

    fc = 400 * 120 + 120 + 120 * 84 + 84 + 84 * 10 + 10
    for name, kinds, nparam in [("LeNet", "SS", 0), ("LeNet-F-I", "SS", 0),
                                ("LeNet-C-alpha", "CC", 1), ("LeNet-C-alpha/beta", "CC", 2),
                                ("LeNet-CM-alpha", "CS", 1), ("LeNet-CM-alpha/beta", "CS", 2),
                                ("LeNet-P-alpha", "PP", 1), ("LeNet-P-alpha/beta", "PP", 2),
                                ("LeNet-PM-alpha", "PS", 1), ("LeNet-PM-alpha/beta", "PS", 2)]:
        total = layer_params(1, 6, kinds[0], nparam) + layer_params(6, 16, kinds[1], nparam) + fc
        assert total == golden[name], name


# ---------------------------------------------------------------- bf16 semantics
def test_bf16_tap_rounding_and_final_rounding():
    """bf16 mode: every tap sum is the exact sum rounded once to bf16 (checked against torch's
    bf16 addition, a library routine), the maximum is exact, y is rounded to bf16."""
    d = inputs.layer(2, 1, 6, 6, 3, 3, 3, stride=1, pad=1, mode="max_plus", dtype="bf16")
    t = inputs.draw(d, 141)
    y = ora.forward(d, t["x"], t["w"])["y"]
    df = dict(d, dtype="f32")
    p = unfold_ref.unfold(df, t["x"])                                   # [N,1,9,OH,OW]
    tb = (torch.from_numpy(p).to(torch.bfloat16)[:, None]
          + torch.from_numpy(t["w"]).to(torch.bfloat16).reshape(1, 3, 1, 9, 1, 1))
    want = tb.float().numpy().max(axis=(2, 3))
    assert same_bits(y, want)
    # a case where fp32 and bf16 rounding differ: 1 + 2^-9 rounds to 1 in bf16
    d1 = inputs.layer(1, 1, 1, 1, 1, 1, 1, mode="max_plus", dtype="bf16")
    one = np.ones((1, 1, 1, 1), np.float32)
    tiny = np.full((1, 1, 1, 1), 2.0 ** -9, np.float32)
    assert ora.forward(d1, one, tiny)["y"].item() == 1.0
    assert ora.forward(d1, one, 3 * tiny)["y"].item() == 1.0 + 2.0 ** -7   # ties-to-even upward
    assert ora.forward(dict(d1, dtype="f32"), one, tiny)["y"].item() == 1.0 + 2.0 ** -9
    # Sum combine accumulates in fp32 and rounds once at the end
    ds = inputs.layer(1, 4, 5, 5, 2, 3, 3, pad=1, mode="compound", dtype="bf16")
    ts = inputs.draw(ds, 142)
    ys = ora.forward(ds, ts["x"], ts["w"], None, ts["alpha"], ts["beta"], ts["bias"])["y"]
    assert np.all((ys.view(np.uint32) & 0xFFFF) == 0)


def _bf16_unfold_forward(d, t):
    """The unfold formulation in bf16, from library routines only: torch bf16 addition for the
    tap sums (one rounding each), numpy min / max / argmin / argmax (first occurrence) over the
    window axis, the channel combine in fp32 in ascending channel order (fused multiply-adds
    emulated in float64: the product of a bf16 value and a float32 is exact there), the bias
    added in fp32 and one conversion of the result to bf16 by torch.  Returns y (bf16 values as
    float32), idx, codes."""
    N, C, K, R, S = d["N"], d["C"], d["K"], d["R"], d["S"]
    OH, OW = unfold_ref.out_hw(d)
    mode, chan = d["mode"], d["chan"]
    if chan == "default":
        chan = {"max_plus": "max", "min_plus": "min"}.get(mode, "sum")
    p = torch.from_numpy(unfold_ref.unfold(dict(d, dtype="f32"), t["x"])).to(torch.bfloat16)   # exact: bf16 values

    def taps(w):
        wr = torch.from_numpy(w).to(torch.bfloat16).reshape(1, K, C, R * S, 1, 1)
        return (p[:, None] + wr).float().numpy()              # [N,K,C,RS,OH,OW], one bf16 rounding per sum

    t1 = taps(t["w"])
    t2 = taps(t["w2"]) if mode == "parallel" else t1
    mn, amn = t1.min(axis=3), t1.argmin(axis=3)
    mx, amx = t2.max(axis=3), t2.argmax(axis=3)
    idx = codes = None
    if mode in ("compound", "parallel"):
        acc = np.zeros((N, K, OH, OW), np.float32)
        for c in range(C):
            a = np.broadcast_to(t["alpha"][None, :, c, None, None], acc.shape)
            b = np.broadcast_to(t["beta"][None, :, c, None, None], acc.shape)
            acc = unfold_ref.fmaf32(a, mn[:, :, c], acc)
            acc = unfold_ref.fmaf32(b, mx[:, :, c], acc)
        codes = (amn | (amx << 4)).astype(np.uint8)
    else:
        m, am = (mn, amn) if mode == "min_plus" else (mx, amx)
        if chan == "sum":
            acc = np.zeros((N, K, OH, OW), np.float32)
            for c in range(C):
                acc = acc + m[:, :, c]                          # float32 adds, channel order
            codes = (am if mode == "min_plus" else (am << 4)).astype(np.uint8)
        else:
            cs = m.argmax(axis=2) if chan == "max" else m.argmin(axis=2)
            acc = np.take_along_axis(m, cs[:, :, None], axis=2)[:, :, 0]
            tap = np.take_along_axis(am, cs[:, :, None], axis=2)[:, :, 0]
            idx = (cs * (R * S) + tap).astype(np.int32)
    acc = acc.astype(np.float32) + t["bias"].astype(np.float32)[None, :, None, None]
    y = torch.from_numpy(np.ascontiguousarray(acc, np.float32)).to(torch.bfloat16).float().numpy()
    return y, idx, codes


@pytest.mark.parametrize("mode,chan", ALL_MODES)
def test_p1_bf16_matches_unfold_formulation(mode, chan):
    """bf16 layers: output bits and winners equal the unfold formulation built from torch's
    bf16 addition and numpy's reductions, on random inputs (rounded tap sums collide often in
    bf16, so ties already occur) and on small integers (ties everywhere)."""
    cases = [dict(), dict(x=("ints", -3, 3), w=("ints", -2, 2), ab=("dyadic", 1, 1), bias=("dyadic", 4, 1))]
    for ci, dist in enumerate(cases):
        for gi, (s, p, dl) in enumerate([(1, 1, 1), (2, 0, 1), (1, 2, 2), (2, 1, 2)]):
            d = inputs.layer(2, 5, 9, 8, 4, 3, 3, stride=s, pad=p, dil=dl, mode=mode, chan=chan, dtype="bf16")
            if min(inputs.output_hw(d)) <= 0:
                continue
            t = inputs.draw(d, 150 + 10 * ci + gi, **dist)
            o = run_fwd(d, t)
            y, idx, codes = _bf16_unfold_forward(d, t)
            assert same_bits(o["y"], y), (mode, chan, dist, s, p, dl)
            if idx is not None:
                assert np.array_equal(o["idx"], idx)
            else:
                mask = 0xFF if mode in ("compound", "parallel") else (0x0F if mode == "min_plus" else 0xF0)
                assert np.array_equal(o["codes"] & mask, codes & mask)
            if ci == 0 and gi == 0:
                # the random case must really contain bf16 ties (else the winner check is idle)
                t1 = torch.from_numpy(unfold_ref.unfold(dict(d, dtype="f32"), t["x"])).to(torch.bfloat16)[:, None] \
                    + torch.from_numpy(t["w"]).to(torch.bfloat16).reshape(1, d["K"], d["C"], 9, 1, 1)
                t1 = t1.float().numpy()
                ext = t1.min(axis=3, keepdims=True) if mode != "max_plus" else t1.max(axis=3, keepdims=True)
                assert ((t1 == ext).sum(axis=3) > 1).any()


def test_output_shape_follows_pytorch_convention():
    for (H, W, R, S, s, p, dl) in itertools.product((7, 10), (8,), (1, 3), (2, 3), (1, 2, 3), (0, 1, 2), (1, 2)):
        d = inputs.layer(1, 1, H, W, 1, R, S, stride=s, pad=p, dil=dl)
        if H + 2 * p < dl * (R - 1) + 1 or W + 2 * p < dl * (S - 1) + 1:
            continue
        ref = F.conv2d(torch.zeros(1, 1, H, W), torch.zeros(1, 1, R, S), stride=s, padding=p, dilation=dl)
        assert tuple(ref.shape[2:]) == ora.output_shape(d) == inputs.output_hw(d)


# ---------------------------------------------------------------- neutral (identity) padding
NEUTRAL_GEOMS = [(1, 1, 1), (2, 1, 1), (1, 2, 1), (1, 2, 2), (2, 1, 2), (1, 4, 2)]


@pytest.mark.parametrize("mode,chan", ALL_MODES)
def test_neutral_padding_matches_unfold_with_identity_fill(mode, chan):
    """pad_mode "neutral": the padding holds the semiring identity (+inf in the min branch, -inf in
    the max branch), so padded taps never win.  Output bits and winners equal the numpy unfold
    formulation whose padding is filled with those infinities."""
    for gi, (s, p, dl) in enumerate(NEUTRAL_GEOMS):
        d = dict(inputs.layer(2, 3, 8, 7, 4, 3, 3, stride=s, pad=p, dil=dl, mode=mode, chan=chan),
                 pad_mode="neutral")
        t = inputs.draw(d, 300 + gi)
        o = run_fwd(d, t)
        two = mode in ("compound", "parallel")
        y, idx, codes = unfold_ref.forward(d, t["x"], t["w"], t["w2"], t["alpha"] if two else None,
                                           t["beta"] if two else None, t["bias"])
        assert np.isfinite(o["y"]).all()
        assert same_bits(o["y"], y), (mode, chan, s, p, dl)
        if idx is not None:
            assert np.array_equal(o["idx"], idx)
        else:
            mask = 0xFF if two else (0x0F if mode == "min_plus" else 0xF0)
            assert np.array_equal(o["codes"] & mask, codes & mask)
        # the Sum forms differ from the zero-padding reading somewhere on the border (a padded tap
        # x = 0 wins some per-channel extremum there)
        if chan == "sum" and gi == 0:
            assert not same_bits(o["y"], run_fwd(dict(d, pad_mode="zero"), t)["y"])


@pytest.mark.parametrize("stride,pad,R", [(1, 1, 3), (2, 1, 3), (1, 1, 2), (3, 1, 3)])
def test_neutral_padding_zero_weight_is_padded_max_pooling(stride, pad, R):
    """w = 0 with neutral padding: MaxPlus-Max is the max over channels of torch's max_pool2d with
    the same padding (which pads with -inf); MinPlus-Min via -x."""
    d = dict(inputs.layer(2, 3, 11, 12, 2, R, R, stride=stride, pad=pad, mode="max_plus"), pad_mode="neutral")
    t = inputs.draw(d, 310)
    w0 = np.zeros_like(t["w"])
    y = ora.forward(d, t["x"], w0)["y"]
    pooled = F.max_pool2d(torch.from_numpy(t["x"]), R, stride=stride, padding=pad).numpy()
    assert same_bits(y, pooled.max(axis=1, keepdims=True).repeat(2, axis=1))
    ymin = ora.forward(dict(d, mode="min_plus"), t["x"], w0)["y"]
    pooled = -F.max_pool2d(torch.from_numpy(-t["x"]), R, stride=stride, padding=pad).numpy()
    assert same_bits(ymin, pooled.min(axis=1, keepdims=True).repeat(2, axis=1))


def test_neutral_padding_constant_input_sees_only_the_valid_taps():
    """x = 0 with neutral padding: every output is the extremum of the weights of the taps that
    lie inside the image (brute force over the window), so border outputs differ from interior
    ones only through which taps are valid."""
    d = dict(inputs.layer(1, 2, 5, 6, 3, 3, 3, stride=1, pad=1, mode="max_plus"), pad_mode="neutral")
    t = inputs.draw(d, 311)
    y = ora.forward(d, np.zeros_like(t["x"]), t["w"])["y"]
    OH, OW = inputs.output_hw(d)
    for k in range(3):
        for oh in range(OH):
            for ow in range(OW):
                vals = [t["w"][k, c, r, s] for c in range(2) for r in range(3) for s in range(3)
                        if 0 <= oh - 1 + r < 5 and 0 <= ow - 1 + s < 6]
                assert y[0, k, oh, ow] == max(vals)


@pytest.mark.parametrize("mode,chan", ALL_MODES)
def test_neutral_padding_backward_loses_nothing_to_the_padding(mode, chan):
    """With neutral padding every winner lies inside the image, so the whole upstream gradient
    reaches grad_x even with pad > 0 (with zero padding the part won by padded taps does not):
    sum(grad_x) = sum_k coefficient * grad_bias[k], exactly on dyadic inputs."""
    d = dict(inputs.layer(2, 3, 6, 7, 4, 3, 3, stride=1, pad=1, mode=mode, chan=chan), pad_mode="neutral")
    t = inputs.draw(d, 312, **DYADIC)
    two = mode in ("compound", "parallel")
    gr = ora.backward(d, t["x"], t["w"], t["g"], t["w2"] if mode == "parallel" else None,
                      t["alpha"] if two else None, t["beta"] if two else None)
    gb = gr["grad_bias"][0]
    if two:
        want = ((t["alpha"] + t["beta"]).astype(np.float64).sum(axis=1) * gb).sum()
    elif chan == "sum":
        want = d["C"] * gb.sum()
    else:
        want = gb.sum()
    assert gr["grad_x"][0].sum() == want
    # the zero-padding reading routes part of the gradient into the padding on these inputs
    gz = ora.backward(dict(d, pad_mode="zero"), t["x"], t["w"], t["g"], t["w2"] if mode == "parallel" else None,
                      t["alpha"] if two else None, t["beta"] if two else None)
    assert not np.array_equal(gz["grad_x"][0], gr["grad_x"][0])


def test_neutral_padding_backward_is_the_directional_derivative():
    """Piecewise linearity with neutral padding: for tie-free inputs and a step that changes no
    winner, the forward difference equals <grad, direction> (float64 arithmetic on the oracle's
    float32 outputs, dyadic grid so that every operation is exact)."""
    d = dict(inputs.layer(1, 2, 5, 5, 2, 3, 3, stride=1, pad=1, mode="compound"), pad_mode="neutral")
    rs = np.random.RandomState(313)
    x = (rs.permutation(50).reshape(1, 2, 5, 5) * 0.25).astype(np.float32)          # distinct, dyadic
    w = (rs.permutation(36).reshape(2, 2, 3, 3) * 16.0).astype(np.float32)          # gaps of 16 > range of x
    al = np.array([[0.5, 1.0], [2.0, -1.0]], np.float32); be = np.array([[1.0, 0.5], [-0.5, 2.0]], np.float32)
    g = rs.randint(-3, 4, (1, 2, 5, 5)).astype(np.float32)
    gr = ora.backward(d, x, w, g, None, al, be)
    u = rs.randint(-2, 3, x.shape).astype(np.float32) * 2.0 ** -6
    y0 = ora.forward(d, x, w, None, al, be)["y"].astype(np.float64)
    y1 = ora.forward(d, x + u, w, None, al, be)["y"].astype(np.float64)
    assert np.array_equal(ora.forward(d, x, w, None, al, be)["codes"], ora.forward(d, x + u, w, None, al, be)["codes"])
    lhs = ((y1 - y0) * g).sum()
    rhs = (gr["grad_x"][0] * u).sum()
    assert lhs == rhs


# ---------------------------------------------------------------- channel statistics
def test_channel_stats_give_numpy_mean_and_variance():
    """The sums the oracle reports reproduce numpy's per-channel mean and (biased) variance, and a
    constant map gives the closed forms count * c and count * c^2."""
    rs = np.random.RandomState(320)
    y = rs.standard_normal((3, 5, 7, 6)).astype(np.float32)
    st = ora.channel_stats(y)
    cnt = 3 * 7 * 6
    mean = st["sum_y"][0] / cnt
    var = st["sum_y2"][0] / cnt - mean ** 2
    assert np.allclose(mean, y.astype(np.float64).mean(axis=(0, 2, 3)), rtol=0, atol=1e-12)
    assert np.allclose(var, y.astype(np.float64).var(axis=(0, 2, 3)), rtol=0, atol=1e-12)
    c = np.full((2, 4, 3, 3), 1.5, np.float32)
    st = ora.channel_stats(c)
    assert np.array_equal(st["sum_y"][0], np.full(4, 18 * 1.5)) and np.array_equal(st["sum_y2"][0], np.full(4, 18 * 2.25))
