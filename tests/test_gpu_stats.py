"""tconv_forward_stats: the forward pass that also returns the per-channel sums of y and y^2 (the
statistics of the batch normalisation that follows a tropical layer).  y and the winners must be
those of tconv_forward bit for bit; the sums are compared with the oracle's float64 sums of the
oracle's y within the summation error bound; the call is deterministic."""
import numpy as np
import pytest
import torch

from oracle import tconv_oracle as ora
from paper_2504_06881_b200 import inputs, tconv
import parity

pytestmark = pytest.mark.gpu

LAYERS = [
    inputs.layer(3, 19, 36, 48, 41, 3, 3, stride=1, pad=1, mode="compound"),                      # copy-engine staging, ragged k tile
    inputs.layer(2, 10, 30, 29, 35, 3, 3, stride=2, pad=1, mode="parallel"),                      # element staging, ragged width
    inputs.layer(2, 7, 28, 28, 9, 3, 3, stride=1, pad=1, mode="max_plus"),                        # ragged pixel tiles
    inputs.layer(4, 16, 14, 14, 24, 3, 3, stride=1, pad=1, mode="compound", dtype="bf16"),
    inputs.layer(2, 12, 24, 32, 20, 3, 3, stride=1, pad=1, mode="min_plus", chan="sum", dtype="bf16"),
    inputs.layer(2, 3, 15, 17, 4, 7, 7, stride=1, pad=3, mode="compound"),                        # any-shape kernel
]


@pytest.mark.parametrize("d", LAYERS, ids=lambda d: f"{d['mode']}-{d['dtype']}-{d['H']}x{d['W']}")
def test_forward_stats_against_the_oracle(d):
    t = inputs.draw(d, 800)
    dev = parity.to_dev(t, d)
    la, ga = parity.layer_args(d, t), parity.layer_args(d, dev)
    y0, win0 = tconv.forward(d, dev["x"], dev["w"], ga["w2"], ga["alpha"], ga["beta"], dev["bias"], want_winners=True)
    y1, win1, s1, s2 = tconv.forward_stats(d, dev["x"], dev["w"], ga["w2"], ga["alpha"], ga["beta"], dev["bias"],
                                           want_winners=True)
    y2, _, r1, r2 = tconv.forward_stats(d, dev["x"], dev["w"], ga["w2"], ga["alpha"], ga["beta"], dev["bias"],
                                        want_winners=True)
    y3, _, q1, q2 = tconv.forward_stats(d, dev["x"], dev["w"], ga["w2"], ga["alpha"], ga["beta"], dev["bias"])
    torch.cuda.synchronize()
    assert torch.equal(y0, y1) and torch.equal(win0, win1) and torch.equal(y0, y3)
    assert torch.equal(s1, r1) and torch.equal(s2, r2)            # the same call twice: identical bits
    # (without winners another kernel variant with another tiling runs: same sums within rounding)
    assert torch.allclose(s1, q1, rtol=1e-5, atol=1e-3) and torch.allclose(s2, q2, rtol=1e-5, atol=1e-3)
    ref = ora.forward(d, t["x"], t["w"], la["w2"], la["alpha"], la["beta"], t["bias"])
    assert parity.same_bits(y1.float().cpu().numpy(), ref["y"]).all()
    st = ora.channel_stats(ref["y"])
    for got, (want, scale) in ((s1, st["sum_y"]), (s2, st["sum_y2"])):
        err = np.abs(got.cpu().numpy().astype(np.float64) - want)
        assert (err <= 1e-5 * scale + 1e-30).all(), (err.max(), scale.max())
