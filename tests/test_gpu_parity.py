"""Parity of the CUDA path (through the C ABI) against the CPU oracle."""
import numpy as np
import pytest
import torch

from paper_2504_06881_b200 import inputs
import parity

pytestmark = pytest.mark.gpu

ALL_MODES = [("max_plus", "max"), ("min_plus", "min"), ("max_plus", "sum"), ("min_plus", "sum"),
             ("max_plus", "min"), ("min_plus", "max"), ("compound", "sum"), ("parallel", "sum")]
TIES = dict(x=("ints", -1, 1), w=("ints", -1, 1))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("mode,chan", ALL_MODES)
def test_small_exhaustive_geometries(mode, chan, dtype):
    """Every stride / pad / dilation in {1,2}x{0,1,2}x{1,2} on maps up to 9x10, random and
    tie-heavy inputs."""
    seed = 0
    for s in (1, 2):
        for p in (0, 1, 2):
            for dl in (1, 2):
                for (H, W, R, S) in ((9, 10, 3, 3), (7, 5, 2, 3)):
                    d = inputs.layer(2, 3, H, W, 5, R, S, stride=s, pad=p, dil=dl, mode=mode,
                                     chan=chan, dtype=dtype)
                    if min(inputs.output_hw(d)) <= 0:
                        continue
                    seed += 1
                    parity.check_layer(d, None, 200 + seed, recompute=(seed % 4 == 0))
                    parity.check_layer(d, TIES, 300 + seed, recompute=False)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_cfg1_compound(dtype):
    """The small benchmark configuration: compound, N=2, C=3, 32x32, K=16, 3x3, pad 1; random
    alpha/beta, the fixed (0.5, 0.5) specialisation, and the parameter-free variant."""
    d, dist = inputs.cfg1()
    d = dict(d, dtype=dtype)
    parity.check_layer(d, dist, 1010)
    t = inputs.draw(d, 1011, **dist)
    t["alpha"][:] = 0.5; t["beta"][:] = 0.5
    parity.check_forward(d, t)
    for mode, chan in ALL_MODES:
        parity.check_layer(dict(d, mode=mode, chan=chan), dist, 1012)


@pytest.mark.parametrize("mode,chan", ALL_MODES)
def test_multi_tile_ragged(mode, chan):
    """Sizes that span several tiles with ragged tails in every dimension."""
    for dtype in ("f32", "bf16"):
        d = inputs.layer(3, 19, 37, 45, 41, 3, 3, stride=1, pad=1, mode=mode, chan=chan, dtype=dtype)
        parity.check_layer(d, None, 401, recompute=False)
    d = inputs.layer(2, 10, 30, 29, 35, 3, 3, stride=2, pad=1, mode=mode, chan=chan)
    parity.check_layer(d, None, 402, recompute=False)
    d = inputs.layer(2, 9, 21, 40, 33, 3, 3, stride=1, pad=2, dil=2, mode=mode, chan=chan, dtype="bf16")
    parity.check_layer(d, dict(x=("relu_normal", 0.0, 1.0), w=("normal", 0.0, 0.05)), 403,
                       recompute=False)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("mode,chan", ALL_MODES)
def test_tma_staged_shapes(mode, chan, dtype):
    """Shapes whose input rows are 16-byte multiples with 'same' padding take the TMA-staged
    kernels: several channel chunks, ragged K and C, partial row tiles, several column tiles,
    stride 2, dilation 2."""
    from paper_2504_06881_b200 import tconv
    mk = lambda *a, **k: inputs.layer(*a, mode=mode, chan=chan, dtype=dtype, **k)
    cases = [mk(3, 19, 20, 32, 41, 3, 3, stride=1, pad=1),
             mk(2, 10, 30, 56, 35, 3, 3, stride=2, pad=1),
             mk(2, 9, 24, 64, 33, 3, 3, stride=1, pad=2, dil=2),
             mk(2, 17, 28, 28, 16, 3, 3, stride=1, pad=1),
             mk(1, 8, 6, 128, 8, 3, 3, stride=1, pad=1),
             mk(1, 5, 9, 40, 8, 3, 3, stride=1, pad=1)]
    for i, d in enumerate(cases):
        t = inputs.draw(d, 450 + i)
        parity.check_forward(d, t, check_winners=False)
        expect_tma = (d["W"] * (4 if dtype == "f32" else 2)) % 16 == 0
        assert ("tma" in tconv.tconv_last_kernel()) == expect_tma, tconv.tconv_last_kernel()
        assert "tiled" in tconv.tconv_last_kernel()
        assert tconv.tconv_device_status() == 0
        parity.check_layer(d, None, 460 + i, recompute=False)
        parity.check_layer(d, TIES, 470 + i, recompute=False, stored_winners=(i == 0))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("mode,chan", ALL_MODES)
def test_ragged_quad_tiles(mode, chan, dtype):
    """Rows of 6 or 7 quads do not divide a warp's 32 lanes: a tile is then 32 consecutive quads of
    the flattened (image, row, quad) space.  Tiles that start in mid-row, cross into the next image
    (second staged block), cover the last partial tile, and maps so small that a tile spans three
    images (per-element staging)."""
    from paper_2504_06881_b200 import tconv
    mk = lambda *a, **k: inputs.layer(*a, mode=mode, chan=chan, dtype=dtype, **k)
    cases = [mk(3, 9, 10, 24, 12, 3, 3, stride=1, pad=1),      # 6 quads per row, 60 per image
             mk(5, 8, 6, 24, 8, 3, 3, stride=1, pad=1),        # 36 quads per image: most tiles cross images
             mk(6, 8, 4, 24, 8, 3, 3, stride=1, pad=1),        # 24 quads per image: a tile spans three
             mk(3, 10, 28, 28, 20, 3, 3, stride=1, pad=1),     # 7 quads per row
             mk(2, 9, 24, 56, 16, 3, 3, stride=2, pad=1),      # stride 2 onto 12 x 28
             mk(2, 9, 14, 24, 16, 3, 3, stride=1, pad=2, dil=2)]
    for i, d in enumerate(cases):
        parity.check_layer(d, None, 480 + i, recompute=False)
        assert "tiled" in tconv.tconv_last_kernel() or "bwd" in tconv.tconv_last_kernel()
        assert tconv.tconv_device_status() == 0
        parity.check_layer(d, TIES, 490 + i, recompute=False)


def test_other_window_sizes():
    """1x1, 1x3, 5x5 (more than 16 taps: wide winner codes), 7x7 windows."""
    for (R, S, pad) in ((1, 1, 0), (1, 3, 1), (5, 5, 2), (7, 7, 3), (4, 4, 1)):
        for mode, chan in (("max_plus", "max"), ("compound", "sum"), ("parallel", "sum"),
                           ("min_plus", "sum")):
            for dtype in ("f32", "bf16"):
                d = inputs.layer(2, 4, 12, 13, 6, R, S, stride=1, pad=pad, mode=mode, chan=chan,
                                 dtype=dtype)
                parity.check_layer(d, None, 500 + R * 10 + S, recompute=False)


def test_no_bias_and_null_alpha_beta():
    d = inputs.layer(2, 5, 10, 11, 7, 3, 3, pad=1, mode="compound")
    t = inputs.draw(d, 601)
    parity.check_forward(d, t, use_bias=False)
    import torch
    from paper_2504_06881_b200 import tconv
    from oracle import tconv_oracle as ora
    g = parity.to_dev(t, d)
    y, _ = tconv.forward(d, g["x"], g["w"], None, None, None, g["bias"])
    ref = ora.forward(d, t["x"], t["w"], None, None, None, t["bias"])
    assert parity.same_bits(y.cpu().numpy(), ref["y"]).all()
    got = tconv.backward(d, g["x"], g["w"], g["g"], None, None, None, None)
    parity.compare_grads(d, got, ora.backward(d, t["x"], t["w"], t["g"]))


def test_single_pixel_and_single_channel_edges():
    for d in (inputs.layer(1, 1, 1, 1, 1, 1, 1, mode="compound"),
              inputs.layer(1, 1, 3, 3, 1, 3, 3, mode="max_plus"),
              inputs.layer(4, 2, 2, 2, 3, 3, 3, pad=1, mode="parallel"),
              inputs.layer(1, 3, 5, 70, 2, 3, 3, pad=1, mode="min_plus", chan="sum")):
        parity.check_layer(d, None, 701)
        parity.check_layer(dict(d, dtype="bf16"), None, 702)


@pytest.mark.parametrize("mode,dist", [("parallel", None), ("max_plus", None), ("min_plus", None),
                                       ("max_plus", dict(x=("ints", -1, 1), w=("ints", -1, 1)))])
def test_backward_is_deterministic(mode, dist):
    """Three runs give the same bits: the Sum forms (private columns, fixed trees) and the Max / Min
    channel combines (row phases, ordered sub-steps, warp-private histograms), random and tie-heavy
    winners, several row bands and column blocks."""
    d = inputs.layer(4, 16, 40, 44, 24, 3, 3, pad=1, mode=mode)
    t = inputs.draw(d, 801, **(dist or {}))
    from paper_2504_06881_b200 import tconv
    g = parity.to_dev(t, d)
    la = parity.layer_args(d, g)
    runs = []
    for _ in range(3):
        _, win = tconv.forward(d, g["x"], g["w"], la["w2"], la["alpha"], la["beta"], g["bias"], want_winners=True)
        out = tconv.backward(d, g["x"], g["w"], g["g"], la["w2"], la["alpha"], la["beta"], win)
        torch.cuda.synchronize()
        runs.append({k: v.clone() for k, v in out.items()})
    for k in runs[0]:
        assert torch.equal(runs[0][k], runs[1][k]) and torch.equal(runs[0][k], runs[2][k]), k
