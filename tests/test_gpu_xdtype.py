"""bf16 layers fed with float x (x_dtype = "f32"): x is rounded to bf16 while it is staged.  The
results must be bit-identical to converting x first and running the plain bf16 layer, in the
forward pass (outputs and winners) and in the backward pass."""
import pytest
import torch

from paper_2504_06881_b200 import inputs, tconv

pytestmark = pytest.mark.gpu

LAYERS = [
    inputs.layer(3, 19, 36, 48, 41, 3, 3, stride=1, pad=1, mode="compound", dtype="bf16"),     # copy-engine shape otherwise
    inputs.layer(2, 10, 28, 28, 35, 3, 3, stride=1, pad=1, mode="parallel", dtype="bf16"),     # 56-byte rows
    inputs.layer(2, 12, 30, 29, 20, 3, 3, stride=2, pad=1, mode="max_plus", dtype="bf16"),     # int32 winners
    inputs.layer(2, 9, 21, 40, 33, 3, 3, stride=1, pad=2, dil=2, mode="min_plus", chan="sum", dtype="bf16"),
    inputs.layer(4, 64, 7, 7, 64, 3, 3, stride=1, pad=1, mode="compound", dtype="bf16"),       # small map, 4 channels per thread
]


@pytest.mark.parametrize("d", LAYERS, ids=lambda d: f"{d['mode']}-{d['H']}x{d['W']}")
def test_float_x_equals_converted_x(d):
    rs = torch.Generator(device="cuda").manual_seed(77)
    N, C, H, W, K = d["N"], d["C"], d["H"], d["W"], d["K"]
    OH, OW = tconv.tconv_output_shape(d)
    x32 = torch.randn(N, C, H, W, device="cuda", generator=rs)
    bf = torch.bfloat16
    w = (0.1 * torch.randn(K, C, 3, 3, device="cuda", generator=rs)).to(bf)
    w2 = (0.1 * torch.randn(K, C, 3, 3, device="cuda", generator=rs)).to(bf)
    al, be = torch.rand(K, C, device="cuda", generator=rs), torch.rand(K, C, device="cuda", generator=rs)
    bias = torch.rand(K, device="cuda", generator=rs)
    g = torch.randn(N, K, OH, OW, device="cuda", generator=rs).to(bf)
    two, par = d["mode"] in ("compound", "parallel"), d["mode"] == "parallel"
    rest = (w, w2 if par else None, al if two else None, be if two else None)
    y0, win0 = tconv.forward(d, x32.to(bf), *rest, bias, want_winners=True)
    g0 = tconv.backward(d, x32.to(bf), w, g, *rest[1:], winners=win0)
    df = dict(d, x_dtype="f32")
    y1, win1 = tconv.forward(df, x32, *rest, bias, want_winners=True)
    assert "tma" not in tconv.tconv_last_kernel()          # the conversion happens in the element-staged path
    g1 = tconv.backward(df, x32, w, g, *rest[1:], winners=win1)
    g2 = tconv.backward(df, x32, w, g, *rest[1:], winners=None)   # winners recomputed from the float x
    torch.cuda.synchronize()
    assert torch.equal(y0, y1) and torch.equal(win0, win1)
    for name in g0:
        assert torch.equal(g0[name], g1[name]), name
        assert torch.equal(g0[name], g2[name]), name


def test_float_x_needs_a_bf16_layer():
    d = dict(inputs.layer(1, 2, 8, 8, 2, 3, 3, pad=1, mode="compound", dtype="f32"), x_dtype="f32")
    with pytest.raises(tconv.TconvError) as e:
        tconv.tconv_output_shape(d)
    assert e.value.status == -1
