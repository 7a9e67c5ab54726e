"""Pins of the three-dimensional oracle against things other than itself: the (pinned)
two-dimensional oracle for windows and volumes of unit extent along one axis, an independent
sliding-window formulation in numpy, torch's max_pool3d, the symmetry of the definition in the
three spatial axes, autograd of a torch formulation for the gradients, and conservation laws."""
import itertools

import numpy as np
import pytest
import torch

from oracle import tconv_oracle as ora2
from oracle import tconv3d_oracle as ora3
from paper_2504_06881_b200 import inputs

MODES = [("max_plus", "default"), ("min_plus", "default"), ("max_plus", "sum"), ("min_plus", "sum"),
         ("max_plus", "min"), ("min_plus", "max"), ("compound", "default"), ("parallel", "default")]


def _args(d, t):
    two, par = d["mode"] in ("compound", "parallel"), d["mode"] == "parallel"
    return dict(w2=t["w2"] if par else None, alpha=t["alpha"] if two else None,
                beta=t["beta"] if two else None)


def _patches(d, x):
    """[N, C, taps, OD, OH, OW]: the zero-padded input seen through every window offset."""
    N, C, D, H, W, T, R, S = (d[k] for k in ("N", "C", "D", "H", "W", "T", "R", "S"))
    (pd, ph, pw), (sd, sh, sw), (dd, dh, dw) = d["pad"], d["stride"], d["dil"]
    OD, OH, OW = inputs.output_dhw(d)
    xp = np.zeros((N, C, D + 2 * pd, H + 2 * ph, W + 2 * pw), np.float32)
    xp[:, :, pd:pd + D, ph:ph + H, pw:pw + W] = x
    p = np.empty((N, C, T * R * S, OD, OH, OW), np.float32)
    for tap, (t, r, s) in enumerate(itertools.product(range(T), range(R), range(S))):
        p[:, :, tap] = xp[:, :, t * dd:t * dd + (OD - 1) * sd + 1:sd,
                          r * dh:r * dh + (OH - 1) * sh + 1:sh, s * dw:s * dw + (OW - 1) * sw + 1:sw]
    return p


def _fmaf32(a, b, c):
    return (a.astype(np.float64) * b.astype(np.float64) + c.astype(np.float64)).astype(np.float32)


def _sliding_forward(d, t):
    """unfold, broadcast-add, library min / max / argmin / argmax, combine over channels."""
    K, C = d["K"], d["C"]
    taps = d["T"] * d["R"] * d["S"]
    mode, chan = d["mode"], ora3.resolved_chan(d)
    p = _patches(d, t["x"])[:, None]                                        # [N,1,C,taps,...]
    t1 = p + t["w"].reshape(1, K, C, taps, 1, 1, 1)
    t2 = p + t["w2"].reshape(1, K, C, taps, 1, 1, 1) if mode == "parallel" else t1
    mn, amn, mx, amx = t1.min(3), t1.argmin(3), t2.max(3), t2.argmax(3)      # [N,K,C,OD,OH,OW]
    idx = codes = None
    if mode in ("compound", "parallel"):
        y = np.zeros(mn[:, :, 0].shape, np.float32)
        for c in range(C):
            a, b = t["alpha"][:, c].reshape(1, K, 1, 1, 1), t["beta"][:, c].reshape(1, K, 1, 1, 1)
            y = _fmaf32(b, mx[:, :, c], _fmaf32(a, mn[:, :, c], y))
        codes = (amn | (amx << 8)).astype(np.uint16)
    else:
        m, am = (mn, amn) if mode == "min_plus" else (mx, amx)
        if chan == "sum":
            y = np.zeros(m[:, :, 0].shape, np.float32)
            for c in range(C):
                y = y + m[:, :, c]
            codes = (am if mode == "min_plus" else am << 8).astype(np.uint16)
        else:
            cw = m.argmax(2) if chan == "max" else m.argmin(2)               # first occurrence
            y = np.take_along_axis(m, cw[:, :, None], 2)[:, :, 0]
            idx = (cw * taps + np.take_along_axis(am, cw[:, :, None], 2)[:, :, 0]).astype(np.int32)
    y = (y + t["bias"].reshape(1, K, 1, 1, 1)).astype(np.float32)
    return y, idx, codes


GEOMS = [dict(stride=1, pad=0, dil=1), dict(stride=(2, 1, 2), pad=(1, 2, 0), dil=1),
         dict(stride=(1, 2, 1), pad=(2, 1, 2), dil=(2, 1, 2)), dict(stride=2, pad=2, dil=1)]


@pytest.mark.parametrize("mode,chan", MODES)
@pytest.mark.parametrize("geom", GEOMS)
def test_forward_is_the_sliding_window_extremum(mode, chan, geom):
    d = inputs.layer3d(2, 3, 6, 7, 5, 4, T=3, R=2, S=3, mode=mode, chan=chan, **geom)
    t = inputs.draw3d(d, 71, ab=("uniform", -1.0, 1.0))
    got = ora3.forward(d, t["x"], t["w"], bias=t["bias"], **_args(d, t))
    y, idx, codes = _sliding_forward(d, t)
    assert np.array_equal(got["y"].view(np.uint32), y.view(np.uint32))
    if idx is not None:
        assert np.array_equal(got["idx"], idx)
    else:
        assert np.array_equal(got["codes"], codes)


def test_ties_go_to_the_lowest_flattened_tap():
    d = inputs.layer3d(1, 3, 5, 5, 5, 2, T=2, R=3, S=2, pad=1, mode="compound")
    t = inputs.draw3d(d, 72, x=("ints", -1, 1), w=("ints", -1, 1))
    got = ora3.forward(d, t["x"], t["w"], bias=t["bias"], **_args(d, t))
    y, _, codes = _sliding_forward(d, t)
    assert np.array_equal(got["codes"], codes) and np.array_equal(got["y"], y)
    d2 = dict(d, mode="max_plus")
    got = ora3.forward(d2, t["x"], t["w"])
    _, idx, _ = _sliding_forward(d2, dict(t, bias=np.zeros(2, np.float32)))
    assert np.array_equal(got["idx"], idx)


@pytest.mark.parametrize("mode,chan", MODES)
@pytest.mark.parametrize("axis", [0, 1, 2])
def test_unit_extent_along_one_axis_is_the_two_dimensional_layer(mode, chan, axis):
    """A volume and window of extent 1 along one axis is a two-dimensional layer: forward and
    backward must agree with the two-dimensional oracle whichever axis is the flat one."""
    size, win, stride, pad, dil = [7, 9], [3, 2], [2, 1], [1, 2], [1, 2]
    full = lambda v, one: tuple(v[:axis] + [one] + v[axis:])
    (D, H, W), (T, R, S) = full(size, 1), full(win, 1)
    d3 = inputs.layer3d(2, 3, D, H, W, 4, T=T, R=R, S=S, stride=full(stride, 1), pad=full(pad, 0),
                        dil=full(dil, 1), mode=mode, chan=chan)
    d2 = ora2.make_desc(2, 3, size[0], size[1], 4, win[0], win[1], stride=tuple(stride), pad=tuple(pad),
                        dil=tuple(dil), mode=mode, chan=chan)
    t = inputs.draw3d(d3, 73, ab=("uniform", -1.0, 1.0))
    sq = lambda a: None if a is None else np.squeeze(a, axis=axis + 2 if a.ndim == 5 else axis + 3)
    kw = _args(d3, t)
    f3 = ora3.forward(d3, t["x"], t["w"], bias=t["bias"], **kw)
    f2 = ora2.forward(d2, sq(t["x"]), sq(t["w"]), w2=sq(kw["w2"]), alpha=kw["alpha"], beta=kw["beta"],
                      bias=t["bias"])
    assert np.array_equal(sq(f3["y"]).view(np.uint32), f2["y"].view(np.uint32))
    if f2["idx"] is not None:
        assert np.array_equal(sq(f3["idx"]), f2["idx"])
    else:
        c3 = sq(f3["codes"])
        assert np.array_equal(((c3 & 0xFF) | ((c3 >> 8) << 4)).astype(np.uint8), f2["codes"])
    b3 = ora3.backward(d3, t["x"], t["w"], t["g"], **kw)
    b2 = ora2.backward(d2, sq(t["x"]), sq(t["w"]), sq(t["g"]), w2=sq(kw["w2"]), alpha=kw["alpha"],
                       beta=kw["beta"])
    assert set(b3) == set(b2)
    for name in b2:
        for i in (0, 1):
            a3 = b3[name][i]
            a3 = sq(a3) if a3.ndim == 5 else a3
            np.testing.assert_allclose(a3, b2[name][i], rtol=1e-12, atol=1e-12, err_msg=name)


@pytest.mark.parametrize("perm", [(0, 2, 1), (1, 0, 2), (2, 1, 0), (1, 2, 0)])
def test_permuting_the_spatial_axes_permutes_the_output(perm):
    d = inputs.layer3d(1, 2, 5, 6, 7, 3, T=2, R=3, S=2, stride=(1, 2, 1), pad=(1, 0, 2), dil=(2, 1, 1),
                       mode="parallel")
    t = inputs.draw3d(d, 74)
    ax = tuple(2 + p for p in perm)
    pick = lambda v: tuple(v[p] for p in perm)
    size, win = pick((d["D"], d["H"], d["W"])), pick((d["T"], d["R"], d["S"]))
    dp = inputs.layer3d(1, 2, *size, 3, T=win[0], R=win[1], S=win[2], stride=pick(d["stride"]),
                        pad=pick(d["pad"]), dil=pick(d["dil"]), mode="parallel")
    tr = lambda a: np.ascontiguousarray(np.transpose(a, (0, 1) + ax))
    y = ora3.forward(d, t["x"], t["w"], bias=t["bias"], **_args(d, t))["y"]
    yp = ora3.forward(dp, tr(t["x"]), tr(t["w"]), w2=tr(t["w2"]), alpha=t["alpha"], beta=t["beta"],
                      bias=t["bias"])["y"]
    assert np.array_equal(tr(y), yp)


def test_zero_weight_max_plus_is_max_pool3d():
    d = inputs.layer3d(2, 1, 8, 9, 10, 1, T=3, R=3, S=3, stride=2, pad=1, mode="max_plus")
    t = inputs.draw3d(d, 75)
    x = np.abs(t["x"])      # non-negative input: zero padding equals max_pool3d's -inf padding
    got = ora3.forward(d, x, np.zeros((1, 1, 3, 3, 3), np.float32))["y"]
    ref = torch.nn.functional.max_pool3d(torch.from_numpy(x), 3, stride=2, padding=1).numpy()
    assert np.array_equal(got, ref)


def test_min_plus_is_negated_max_plus_and_weight_shift_shifts_the_output():
    d = inputs.layer3d(2, 3, 5, 6, 5, 4, T=2, R=2, S=3, pad=1, mode="min_plus", chan="sum")
    t = inputs.draw3d(d, 76)
    mn = ora3.forward(d, t["x"], t["w"])["y"]
    mx = ora3.forward(dict(d, mode="max_plus"), -t["x"], -t["w"])["y"]
    assert np.array_equal(mn, -mx)
    dy = inputs.layer3d(1, 1, 4, 4, 4, 1, T=2, R=2, S=2, mode="max_plus")
    td = inputs.draw3d(dy, 77, x=("dyadic", 6, 2), w=("dyadic", 6, 2))
    base = ora3.forward(dy, td["x"], td["w"])["y"]
    assert np.array_equal(ora3.forward(dy, td["x"], td["w"] + np.float32(0.75))["y"], base + np.float32(0.75))
    d1 = inputs.layer3d(2, 1, 3, 4, 5, 1, T=1, R=1, S=1, mode="min_plus")
    t1 = inputs.draw3d(d1, 78)
    assert np.array_equal(ora3.forward(d1, t1["x"], t1["w"])["y"], t1["x"] + t1["w"].reshape(()))


@pytest.mark.parametrize("mode,chan", MODES)
def test_gradients_match_autograd_of_a_torch_formulation(mode, chan):
    """torch (float64): pad, unfold the three axes, add, amin / amax, combine; autograd routes
    the gradient to the winner when there are no ties (continuous random data)."""
    d = inputs.layer3d(2, 3, 6, 5, 7, 4, T=2, R=3, S=2, stride=(1, 2, 1), pad=(1, 1, 0), mode=mode, chan=chan)
    t = inputs.draw3d(d, 79, ab=("uniform", -1.0, 1.0))
    two, par = mode in ("compound", "parallel"), mode == "parallel"
    T64 = lambda a: torch.from_numpy(a.astype(np.float64)).requires_grad_(True)
    x, w, w2, al, be, bias = (T64(t[k]) for k in ("x", "w", "w2", "alpha", "beta", "bias"))
    pd, ph, pw = d["pad"]
    xp = torch.nn.functional.pad(x, (pw, pw, ph, ph, pd, pd))
    u = xp.unfold(2, d["T"], d["stride"][0]).unfold(3, d["R"], d["stride"][1]).unfold(4, d["S"], d["stride"][2])
    u = u.reshape(*u.shape[:5], -1)[:, None]                                  # [N,1,C,OD,OH,OW,taps]
    wv = lambda a: a.reshape(1, d["K"], d["C"], 1, 1, 1, -1)
    mn, mx = (u + wv(w)).amin(-1), (u + wv(w2 if par else w)).amax(-1)        # [N,K,C,OD,OH,OW]
    cw = lambda a: a.reshape(1, d["K"], d["C"], 1, 1, 1)
    if two:
        y = (cw(al) * mn + cw(be) * mx).sum(2)
    else:
        m = mn if mode == "min_plus" else mx
        rc = ora3.resolved_chan(d)
        y = m.sum(2) if rc == "sum" else (m.amax(2) if rc == "max" else m.amin(2))
    y = y + bias.reshape(1, -1, 1, 1, 1)
    y.backward(torch.from_numpy(t["g"].astype(np.float64)))
    got = ora3.backward(d, t["x"], t["w"], t["g"], **_args(d, t))
    ref = {"grad_x": x.grad, "grad_w": w.grad, "grad_bias": bias.grad}
    if par:
        ref["grad_w2"] = w2.grad
    if two:
        ref["grad_alpha"], ref["grad_beta"] = al.grad, be.grad
    assert set(got) == set(ref)
    for name, r in ref.items():
        np.testing.assert_allclose(got[name][0], r.numpy(), rtol=1e-6, atol=1e-6, err_msg=name)
        assert np.all(got[name][1] + 1e-12 >= np.abs(got[name][0]))


def test_gradient_conservation_without_padding():
    d = inputs.layer3d(2, 3, 6, 6, 6, 4, T=3, R=3, S=3, mode="max_plus")
    t = inputs.draw3d(d, 80)
    b = ora3.backward(d, t["x"], t["w"], t["g"])
    total = t["g"].astype(np.float64).sum()
    for name in ("grad_x", "grad_w", "grad_bias"):
        assert abs(b[name][0].sum() - total) < 1e-9
    dc = dict(d, mode="compound")
    bc = ora3.backward(dc, t["x"], t["w"], t["g"], alpha=t["alpha"], beta=t["beta"])
    per_k = t["g"].astype(np.float64).sum(axis=(0, 2, 3, 4))
    want = ((t["alpha"].astype(np.float64) + t["beta"]) * per_k[:, None]).sum()
    assert abs(bc["grad_x"][0].sum() - want) < 1e-8 and abs(bc["grad_w"][0].sum() - want) < 1e-8


@pytest.mark.parametrize("mode,chan", MODES)
def test_one_dimensional_layers_with_long_windows(mode, chan):
    """Unit depth and height with a 1 x 1 x 80 window at stride 4 (the opening layer of the paper's
    audio networks) against a formulation written out in one dimension with numpy's strided
    windows, and against the (pinned) two-dimensional oracle on a signal of unit height."""
    d = inputs.layer3d(2, 3, 1, 1, 413, 4, T=1, R=1, S=80, stride=(1, 1, 4), pad=(0, 0, 9), mode=mode, chan=chan)
    t = inputs.draw3d(d, 4242, x=("ints", -3, 3), w=("ints", -2, 2)) if chan in ("min", "max") else inputs.draw3d(d, 4242)
    out = ora3.forward(d, t["x"], t["w"], bias=t["bias"], **_args(d, t))
    N, C, K, S, L = d["N"], d["C"], d["K"], 80, 413
    xp = np.zeros((N, C, L + 18), np.float32)
    xp[:, :, 9:9 + L] = t["x"][:, :, 0, 0]
    win = np.lib.stride_tricks.sliding_window_view(xp, S, axis=2)[:, :, ::4]          # [N, C, OL, S]
    t1 = win[:, None] + t["w"].reshape(1, K, C, 1, S)                                 # [N, K, C, OL, S]
    t2 = win[:, None] + t["w2"].reshape(1, K, C, 1, S) if mode == "parallel" else t1
    mn, mx = t1.min(-1), t2.max(-1)
    if mode in ("compound", "parallel"):
        y = np.zeros(mn[:, :, 0].shape, np.float32)
        for c in range(C):
            y = _fmaf32(t["beta"][:, c].reshape(1, K, 1), mx[:, :, c], _fmaf32(t["alpha"][:, c].reshape(1, K, 1), mn[:, :, c], y))
        assert np.array_equal(out["codes"][:, :, :, 0, 0], (t1.argmin(-1) | (t2.argmax(-1) << 8)).astype(np.uint16))
    else:
        m = mn if mode == "min_plus" else mx
        rc = ora3.resolved_chan(d)
        if rc == "sum":
            y = np.zeros(m[:, :, 0].shape, np.float32)
            for c in range(C):
                y = (y + m[:, :, c]).astype(np.float32)
        else:
            y = m.max(2) if rc == "max" else m.min(2)
    y = (y + t["bias"].reshape(1, K, 1)).astype(np.float32)
    assert np.array_equal(out["y"][:, :, 0, 0], y)
    # the same layer as a 1 x 80 window on a signal of unit height, through the two-dimensional oracle
    d2 = inputs.layer(2, 3, 1, 413, 4, 1, 80, stride=(1, 4), pad=(0, 9), mode=mode, chan=chan)
    two, par = mode in ("compound", "parallel"), mode == "parallel"
    ref = ora2.forward(d2, t["x"][:, :, 0], t["w"][:, :, 0], t["w2"][:, :, 0] if par else None,
                       t["alpha"] if two else None, t["beta"] if two else None, t["bias"])
    assert np.array_equal(out["y"][:, :, 0], ref["y"])
    g3 = ora3.backward(d, t["x"], t["w"], t["g"], **_args(d, t))
    g2 = ora2.backward(d2, t["x"][:, :, 0], t["w"][:, :, 0], t["g"][:, :, 0], t["w2"][:, :, 0] if par else None,
                       t["alpha"] if two else None, t["beta"] if two else None)
    for k in g2:
        assert np.allclose(np.asarray(g3[k]).reshape(np.asarray(g2[k]).shape), g2[k], rtol=1e-6, atol=1e-6), k
