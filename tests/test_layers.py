"""The named layer set (Section 3.1 layers (i)-(vi), compound / parallel with 0p / 1p / 2p scalars,
the alpha / beta specialisations of the paper's section
"Specializations of compound/parallel tropical convolutions")."""
from pathlib import Path

import numpy as np
import pytest
import torch

from paper_2504_06881_b200 import inputs, layers


def _golden():
    out = {}
    for line in (Path(__file__).parent / "golden" / "lenet_param_counts.txt").read_text().splitlines():
        if line and not line.startswith("#"):
            name, n = line.split()
            out[name] = int(n)
    return out


def test_lenet_variants_built_from_the_named_layers_have_the_papers_parameter_counts():
    """LeNet: conv 1->6 5x5, conv 6->16 5x5, fc 400-120-84-10 (results table of the LeNet section).
    C / P = both convolutions compound / parallel, CM / PM = only the first one."""
    import torch.nn as nn
    g = _golden()
    fc = 400 * 120 + 120 + 120 * 84 + 84 + 84 * 10 + 10
    count = lambda *mods: sum(p.numel() for m in mods for p in m.parameters()) + fc
    std = lambda ci, co: nn.Conv2d(ci, co, 5)
    C1, C2 = layers.CompoundMinMaxPlusSumConv2d1p, layers.CompoundMinMaxPlusSumConv2d2p
    P1, P2 = layers.ParallelMinMaxPlusSumConv2d1p, layers.ParallelMinMaxPlusSumConv2d2p
    assert count(std(1, 6), std(6, 16)) == g["LeNet"]
    assert count(layers.MinPlusSumConv2d(1, 6, 5), layers.MaxPlusSumConv2d(6, 16, 5)) == g["LeNet-F-I"]
    assert count(C1(1, 6, 5), C1(6, 16, 5)) == g["LeNet-C-alpha"]
    assert count(C2(1, 6, 5), C2(6, 16, 5)) == g["LeNet-C-alpha/beta"]
    assert count(C1(1, 6, 5), std(6, 16)) == g["LeNet-CM-alpha"]
    assert count(C2(1, 6, 5), std(6, 16)) == g["LeNet-CM-alpha/beta"]
    assert count(P1(1, 6, 5), P1(6, 16, 5)) == g["LeNet-P-alpha"]
    assert count(P2(1, 6, 5), P2(6, 16, 5)) == g["LeNet-P-alpha/beta"]
    assert count(P1(1, 6, 5), std(6, 16)) == g["LeNet-PM-alpha"]
    assert count(P2(1, 6, 5), std(6, 16)) == g["LeNet-PM-alpha/beta"]


def test_names_map_to_modes_and_channel_combines():
    table = {"MaxPlusSumConv2d": ("max_plus", "sum"), "MinPlusSumConv2d": ("min_plus", "sum"),
             "MinPlusMaxConv2d": ("min_plus", "max"), "MinPlusMinConv2d": ("min_plus", "min"),
             "MaxPlusMaxConv2d": ("max_plus", "max"), "MaxPlusMinConv2d": ("max_plus", "min")}
    for name, (mode, chan) in table.items():
        m = getattr(layers, name)(3, 4, 3, padding=1)
        assert (m.mode, m.chan) == (mode, chan)
        assert m.alpha is None and m.beta is None and m.weight2 is None
    for fam, mode in (("Compound", "compound"), ("Parallel", "parallel")):
        for np_, (has_a, has_b) in (("0p", (False, False)), ("1p", (True, False)), ("2p", (True, True))):
            m = getattr(layers, f"{fam}MinMaxPlusSumConv2d{np_}")(3, 4, 3)
            assert m.mode == mode and m.params == np_
            assert (m.alpha is not None, m.beta is not None) == (has_a, has_b)
            assert (m.weight2 is not None) == (mode == "parallel")
    with pytest.raises(ValueError):
        layers.TropicalConv2d(3, 4, 3, params="3p")


@pytest.mark.gpu
@pytest.mark.parametrize("mode", ["compound", "parallel"])
@pytest.mark.parametrize("params", ["0p", "1p", "2p", "shared", "opposite", "fixed"])
def test_specialisations_against_the_oracle(mode, params):
    """Forward bit-exact and the chained alpha gradient (beta = f(alpha)) against the oracle run
    with the alpha / beta arrays the specialisation implies."""
    from oracle import tconv_oracle as ora
    d = inputs.layer(2, 5, 9, 12, 7, 3, 3, stride=1, pad=1, mode=mode)
    t = inputs.draw(d, 2100)
    m = layers.TropicalConv2d(5, 7, 3, padding=1, mode=mode, params=params, fixed=(1.0, -1.0)).cuda()
    with torch.no_grad():
        m.weight.copy_(torch.from_numpy(t["w"]))
        m.bias.copy_(torch.from_numpy(t["bias"]))
        if m.weight2 is not None:
            m.weight2.copy_(torch.from_numpy(t["w2"]))
        if m.alpha is not None:
            m.alpha.copy_(torch.from_numpy(t["alpha"]))
        if m.beta is not None:
            m.beta.copy_(torch.from_numpy(t["beta"]))
    a = t["alpha"]
    ab = {"0p": (np.ones_like(a), np.ones_like(a)), "1p": (a, (1.0 - torch.from_numpy(a)).numpy()), "2p": (a, t["beta"]),
          "shared": (a, a), "opposite": (a, -a),
          "fixed": (np.full_like(a, 1.0), np.full_like(a, -1.0))}[params]
    w2 = t["w2"] if mode == "parallel" else None
    ref = ora.forward(d, t["x"], t["w"], w2, ab[0], ab[1], t["bias"])
    x = torch.from_numpy(t["x"]).cuda().requires_grad_(True)
    y = m(x)
    assert np.array_equal(y.detach().cpu().numpy().view(np.uint32), ref["y"].view(np.uint32))
    y.backward(torch.from_numpy(t["g"]).cuda())
    gref = ora.backward(d, t["x"], t["w"], t["g"], w2, ab[0], ab[1])   # name -> (gradient, sum of |contributions|)

    def close(got, want, scale):
        return (np.abs(got.detach().cpu().numpy().astype(np.float64) - want) <= 1e-5 * scale + 1e-30).all()

    assert close(x.grad, *gref["grad_x"])
    assert close(m.weight.grad, *gref["grad_w"])
    if m.weight2 is not None:
        assert close(m.weight2.grad, *gref["grad_w2"])
    (ga, gaa), (gb, gba) = gref["grad_alpha"], gref["grad_beta"]
    if m.alpha is not None:
        # beta = f(alpha): d loss / d alpha = grad_alpha + f'(alpha) * grad_beta
        sign = {"1p": -1.0, "2p": 0.0, "shared": 1.0, "opposite": -1.0}[params]
        assert close(m.alpha.grad, ga + sign * gb, gaa + abs(sign) * gba)
    if m.beta is not None:
        assert close(m.beta.grad, gb, gba)


@pytest.mark.gpu
@pytest.mark.parametrize("mode,params", [("compound", "2p"), ("compound", "1p"), ("parallel", "2p"), ("max_plus", "0p")])
def test_depthwise_layer_against_the_oracle(mode, params):
    from oracle import tconv_oracle as ora
    from paper_2504_06881_b200.nn import TropicalDepthwiseConv2d
    C = 6
    d = inputs.layer(2, C, 10, 12, C, 3, 3, stride=1, pad=1, mode=mode)
    rs = np.random.RandomState(2200)
    x = rs.standard_normal((2, C, 10, 12)).astype(np.float32)
    g = rs.standard_normal((2, C, 10, 12)).astype(np.float32)
    m = TropicalDepthwiseConv2d(C, 3, padding=1, mode=mode, params=params).cuda()
    two, par = mode in ("compound", "parallel"), mode == "parallel"
    with torch.no_grad():
        if m.alpha is not None:
            m.alpha.copy_(torch.from_numpy(rs.uniform(0, 1, C).astype(np.float32)))
        if m.beta is not None:
            m.beta.copy_(torch.from_numpy(rs.uniform(0, 1, C).astype(np.float32)))
        m.bias.copy_(torch.from_numpy(rs.uniform(-0.1, 0.1, C).astype(np.float32)))
    w = m.weight.detach().cpu().numpy()
    w2 = m.weight2.detach().cpu().numpy() if par else None
    a = m.alpha.detach().cpu().numpy() if m.alpha is not None else None
    b = (m.beta.detach().cpu().numpy() if m.beta is not None else (1.0 - torch.from_numpy(a)).numpy() if params == "1p" else None)
    bias = m.bias.detach().cpu().numpy()
    ref = ora.depthwise_forward(d, x, w, w2, a if two else None, b if two else None, bias)
    xt = torch.from_numpy(x).cuda().requires_grad_(True)
    y = m(xt)
    assert np.array_equal(y.detach().cpu().numpy().view(np.uint32), ref["y"].view(np.uint32))
    y.backward(torch.from_numpy(g).cuda())
    gref = ora.depthwise_backward(d, x, w, g, w2, a if two else None, b if two else None)

    def close(got, want, scale):
        return (np.abs(got.detach().cpu().numpy().astype(np.float64) - want) <= 1e-5 * scale + 1e-30).all()

    assert close(xt.grad, *gref["grad_x"]) and close(m.weight.grad, *gref["grad_w"]) and close(m.bias.grad, *gref["grad_bias"])
    if par:
        assert close(m.weight2.grad, *gref["grad_w2"])
    if m.alpha is not None:
        (ga, gaa), (gb, gba) = gref["grad_alpha"], gref["grad_beta"]
        sign = -1.0 if params == "1p" else 0.0
        assert close(m.alpha.grad, ga + sign * gb, gaa + abs(sign) * gba)
    if m.beta is not None:
        assert close(m.beta.grad, *gref["grad_beta"])


@pytest.mark.gpu
@pytest.mark.parametrize("mode,chan", [("compound", "default"), ("parallel", "default"), ("max_plus", "default"),
                                       ("min_plus", "sum")])
@pytest.mark.parametrize("S,st,pad", [(80, 4, 38), (3, 1, 1)])
def test_conv1d_against_the_oracle(mode, chan, S, st, pad):
    """Kernel length 80, stride 4 (the first layer of the paper's 1-D audio networks) and the length-3
    layers that follow it, against the 2-D oracle on a signal of unit height."""
    from oracle import tconv_oracle as ora
    from paper_2504_06881_b200.nn import TropicalConv1d
    N, C, K, Ln = 2, 3, 5, 400
    d = inputs.layer(N, C, 1, Ln, K, 1, S, stride=(1, st), pad=(0, pad), mode=mode, chan=chan)
    t = inputs.draw(d, 2300)
    m = TropicalConv1d(C, K, S, stride=st, padding=pad, mode=mode, chan=chan).cuda()
    assert m.tiled == (S == 3)
    two, par = mode in ("compound", "parallel"), mode == "parallel"
    with torch.no_grad():
        m.conv.weight.copy_(torch.from_numpy(t["w"]).reshape(m.conv.weight.shape))
        m.conv.bias.copy_(torch.from_numpy(t["bias"]))
        if par:
            m.conv.weight2.copy_(torch.from_numpy(t["w2"]).reshape(m.conv.weight.shape))
        if two:
            m.conv.alpha.copy_(torch.from_numpy(t["alpha"]))
            m.conv.beta.copy_(torch.from_numpy(t["beta"]))
    ref = ora.forward(d, t["x"], t["w"], t["w2"] if par else None, t["alpha"] if two else None,
                      t["beta"] if two else None, t["bias"])
    x = torch.from_numpy(t["x"][:, :, 0]).cuda().requires_grad_(True)
    y = m(x)
    assert np.array_equal(y.detach().cpu().numpy().view(np.uint32), ref["y"][:, :, 0].view(np.uint32))
    y.backward(torch.from_numpy(t["g"][:, :, 0]).cuda())
    gref = ora.backward(d, t["x"], t["w"], t["g"], t["w2"] if par else None, t["alpha"] if two else None,
                        t["beta"] if two else None)

    def close(got, want, scale):
        return (np.abs(got.detach().cpu().numpy().astype(np.float64) - want) <= 1e-5 * scale + 1e-30).all()

    assert close(x.grad.unsqueeze(2), *gref["grad_x"]) and close(m.conv.weight.grad.reshape(K, C, 1, S), *gref["grad_w"])
    if two:
        assert close(m.conv.alpha.grad, *gref["grad_alpha"]) and close(m.conv.beta.grad, *gref["grad_beta"])


def test_conv3d_names_and_lenet3d_parameter_counts():
    """3d:[5/6,2] -> pool -> 3d:[5/16] -> pool (Table 1, configuration 3d): the tropical layers of
    the compound 2p variant hold the weights plus one (alpha, beta) pair per channel pair."""
    c1 = layers.CompoundMinMaxPlusSumConv3d2p(1, 6, 5, stride=2)
    c2 = layers.ParallelMinMaxPlusSumConv3d1p(6, 16, 5)
    count = lambda m: sum(p.numel() for p in m.parameters())
    assert count(c1) == 6 * 125 + 2 * 6 + 6
    assert count(c2) == 2 * 16 * 6 * 125 + 16 * 6 + 16
    assert (layers.MinPlusMaxConv3d(2, 3, 3).mode, layers.MinPlusMaxConv3d(2, 3, 3).chan) == ("min_plus", "max")
    assert layers.MaxPlusSumConv3d(2, 3, (1, 2, 3)).weight.shape == (3, 2, 1, 2, 3)


@pytest.mark.gpu
@pytest.mark.parametrize("mode,params", [("compound", "2p"), ("compound", "1p"), ("parallel", "2p"), ("min_plus", "0p")])
def test_conv3d_layer_against_the_oracle(mode, params):
    from oracle import tconv3d_oracle as ora3
    from paper_2504_06881_b200.nn import TropicalConv3d
    N, C, K = 2, 3, 4
    d = inputs.layer3d(N, C, 9, 8, 10, K, T=3, R=3, S=3, stride=(2, 1, 1), pad=1, mode=mode)
    t = inputs.draw3d(d, 2400, ab=("uniform", -1.0, 1.0))
    m = TropicalConv3d(C, K, 3, stride=(2, 1, 1), padding=1, mode=mode, params=params).cuda()
    two, par = mode in ("compound", "parallel"), mode == "parallel"
    with torch.no_grad():
        m.weight.copy_(torch.from_numpy(t["w"]))
        m.bias.copy_(torch.from_numpy(t["bias"]))
        if par:
            m.weight2.copy_(torch.from_numpy(t["w2"]))
        if two:
            m.alpha.copy_(torch.from_numpy(t["alpha"]))
            if params == "2p":
                m.beta.copy_(torch.from_numpy(t["beta"]))
    beta = t["beta"] if params == "2p" else (1.0 - t["alpha"]).astype(np.float32)
    kw = dict(w2=t["w2"] if par else None, alpha=t["alpha"] if two else None, beta=beta if two else None)
    ref = ora3.forward(d, t["x"], t["w"], bias=t["bias"], **kw)
    x = torch.from_numpy(t["x"]).cuda().requires_grad_(True)
    y = m(x)
    assert np.array_equal(y.detach().cpu().numpy().view(np.uint32), ref["y"].view(np.uint32))
    y.backward(torch.from_numpy(t["g"]).cuda())
    gref = ora3.backward(d, t["x"], t["w"], t["g"], **kw)

    def close(got, want, scale):
        return (np.abs(got.detach().cpu().numpy().astype(np.float64) - want) <= 1e-5 * scale + 1e-30).all()

    assert close(x.grad, *gref["grad_x"]) and close(m.weight.grad, *gref["grad_w"])
    assert close(m.bias.grad, *gref["grad_bias"])
    if par:
        assert close(m.weight2.grad, *gref["grad_w2"])
    if two and params == "2p":
        assert close(m.alpha.grad, *gref["grad_alpha"]) and close(m.beta.grad, *gref["grad_beta"])
    if two and params == "1p":       # beta = 1 - alpha: the chain rule gives grad_alpha - grad_beta
        want = gref["grad_alpha"][0] - gref["grad_beta"][0]
        assert close(m.alpha.grad, want, gref["grad_alpha"][1] + gref["grad_beta"][1])
    # a first layer: the input needs no gradient and none is computed
    y2 = m(torch.from_numpy(t["x"]).cuda())
    y2.sum().backward()
