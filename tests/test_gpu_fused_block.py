"""The residual block with the layer's fused extras: batch-normalisation statistics taken in the
tropical kernels' epilogue (tconv_forward_stats) and float activations read by the bf16 kernels
directly (x_dtype).  Both must leave the block's results unchanged up to rounding: compared with
the plain block (separate cast kernels, torch batch normalisation) on the same parameters."""
import copy

import pytest
import torch

from paper_2504_06881_b200.nn import TropicalBasicBlock, TropicalConvFn

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("mode", ["compound", "parallel"])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_fused_block_matches_the_plain_block(mode, dtype):
    torch.manual_seed(5)
    plain = TropicalBasicBlock(16, 24, 2, mode, dtype).cuda().train()
    fused = copy.deepcopy(plain)
    fused.fused_bn = True
    x = torch.randn(4, 16, 28, 28, device="cuda")
    g = torch.randn(4, 24, 14, 14, device="cuda")
    outs = []
    for blk, cast in ((plain, False), (fused, True)):
        TropicalConvFn.fuse_cast = cast
        xi = x.clone().requires_grad_(True)
        y = blk(xi)
        y.backward(g)
        outs.append((y.detach(), xi.grad.detach(), {n: p.grad.detach() for n, p in blk.named_parameters()},
                     blk.bn1.running_mean.clone(), blk.bn2.running_var.clone()))
    TropicalConvFn.fuse_cast = False
    (y0, gx0, gp0, rm0, rv0), (y1, gx1, gp1, rm1, rv1) = outs
    tol = dict(rtol=2e-3, atol=2e-3) if dtype == "f32" else dict(rtol=5e-2, atol=5e-2)
    assert torch.allclose(y0, y1, **tol)
    assert torch.allclose(rm0, rm1, rtol=1e-4, atol=1e-5) and torch.allclose(rv0, rv1, rtol=1e-3, atol=1e-5)
    assert torch.allclose(gx0, gx1, **tol)
    for n in gp0:
        scale = gp0[n].abs().max().item() + 1e-6
        assert (gp0[n] - gp1[n]).abs().max().item() <= (5e-3 if dtype == "f32" else 8e-2) * scale, n


def test_float_x_path_is_bit_identical_in_the_layer():
    from paper_2504_06881_b200.nn import TropicalConv2d
    torch.manual_seed(6)
    layer = TropicalConv2d(12, 20, 3, padding=1, mode="compound", dtype="bf16").cuda()
    x = torch.randn(3, 12, 20, 24, device="cuda")
    res = []
    for cast in (False, True):
        TropicalConvFn.fuse_cast = cast
        xi = x.clone().requires_grad_(True)
        y = layer(xi)
        y.backward(torch.ones_like(y))
        res.append((y.detach().clone(), xi.grad.clone(), layer.weight.grad.clone()))
        layer.zero_grad()
    TropicalConvFn.fuse_cast = False
    for a, b in zip(*res):
        assert torch.equal(a, b)
