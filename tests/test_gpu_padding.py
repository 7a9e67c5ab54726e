"""Neutral (semiring-identity) padding on the GPU against the oracle's second padding reading:
padded taps never take part in min / max.  Covers the TMA-staged and the element-staged tiled
kernels in both dtypes, the any-shape kernels, winners, and the backward pass with stored and
with recomputed winners."""
import numpy as np
import pytest
import torch

from paper_2504_06881_b200 import inputs, tconv
import parity

pytestmark = pytest.mark.gpu

ALL_MODES = [("max_plus", "max"), ("min_plus", "min"), ("max_plus", "sum"), ("min_plus", "sum"),
             ("max_plus", "min"), ("min_plus", "max"), ("compound", "sum"), ("parallel", "sum")]
TIES = dict(x=("ints", -1, 1), w=("ints", -1, 1))


def neutral(d):
    return dict(d, pad_mode="neutral")


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("mode,chan", ALL_MODES)
def test_neutral_padding_small_geometries(mode, chan, dtype):
    seed = 0
    for (s, p, dl) in ((1, 1, 1), (2, 1, 1), (1, 2, 2), (2, 2, 2), (1, 2, 1), (1, 4, 2)):
        for (H, W, R, S) in ((9, 10, 3, 3), (7, 5, 2, 3)):
            if p > (R - 1) * dl or p > (S - 1) * dl:
                continue
            d = neutral(inputs.layer(2, 3, H, W, 5, R, S, stride=s, pad=p, dil=dl, mode=mode, chan=chan, dtype=dtype))
            seed += 1
            parity.check_layer(d, None, 500 + seed, recompute=(seed % 3 == 0))
            parity.check_layer(d, TIES, 600 + seed, recompute=False)


@pytest.mark.parametrize("mode,chan", ALL_MODES)
def test_neutral_padding_multi_tile(mode, chan):
    """Tiled kernels on several tiles: copy-engine staging (rows that are 16-byte multiples, "same"
    padding), element staging (other widths / paddings), stride 2, dilation 2, both dtypes."""
    for dtype in ("f32", "bf16"):
        d = neutral(inputs.layer(3, 19, 36, 48, 41, 3, 3, stride=1, pad=1, mode=mode, chan=chan, dtype=dtype))
        parity.check_forward(d, inputs.draw(d, 701))
        assert "tma" in tconv.tconv_last_kernel()
        parity.check_layer(d, None, 701, recompute=False)
        d = neutral(inputs.layer(2, 10, 30, 29, 35, 3, 3, stride=2, pad=1, mode=mode, chan=chan, dtype=dtype))
        parity.check_layer(d, None, 702, recompute=False)
    d = neutral(inputs.layer(2, 9, 21, 40, 33, 3, 3, stride=1, pad=2, dil=2, mode=mode, chan=chan, dtype="bf16"))
    parity.check_layer(d, dict(x=("relu_normal", 0.0, 1.0), w=("normal", 0.0, 0.05)), 703, recompute=False)
    d = neutral(inputs.layer(2, 6, 28, 28, 20, 3, 3, stride=1, pad=1, mode=mode, chan=chan, dtype="bf16"))
    parity.check_layer(d, None, 704, recompute=True)


def test_neutral_padding_any_shape_kernels():
    """Windows the tiled kernels do not serve (7 x 7, stride 3)."""
    for mode, chan in (("compound", "sum"), ("max_plus", "max"), ("min_plus", "sum")):
        d = neutral(inputs.layer(2, 3, 15, 17, 4, 7, 7, stride=1, pad=3, mode=mode, chan=chan))
        parity.check_forward(d, inputs.draw(d, 710))
        assert "generic" in tconv.tconv_last_kernel()
        parity.check_layer(d, None, 710, recompute=False)
        d = neutral(inputs.layer(2, 4, 14, 13, 5, 3, 3, stride=3, pad=1, mode=mode, chan=chan))
        parity.check_layer(d, None, 711, recompute=False)


def test_neutral_padding_is_refused_where_a_window_would_be_empty():
    """pad > (R - 1) * dilation leaves border windows without a tap inside the image."""
    d = neutral(inputs.layer(1, 1, 6, 6, 1, 1, 1, pad=1, mode="max_plus"))
    x = torch.zeros(1, 1, 6, 6, device="cuda"); w = torch.zeros(1, 1, 1, 1, device="cuda")
    with pytest.raises(tconv.TconvError) as e:
        tconv.forward(d, x, w)
    assert e.value.status == -2
