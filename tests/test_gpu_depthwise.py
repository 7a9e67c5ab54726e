"""Parity of the depthwise (groups = C) kernels with the oracle, which applies the dense
single-channel operator channel by channel: forward and winner codes bit for bit, gradients
within the tolerance of the dense layers."""
import numpy as np
import pytest
import torch

from oracle import tconv_oracle as ora
from paper_2504_06881_b200 import inputs, tconv
import parity

pytestmark = pytest.mark.gpu

MODES = ["max_plus", "min_plus", "compound", "parallel"]


def draw(d, seed, ties=False):
    rs = np.random.RandomState(seed)
    N, C, H, W, R, S = (d[k] for k in "NCHWRS")
    OH, OW = ora.output_shape(d)
    if ties:    # small integers: constant ties between taps
        f = lambda *sh: rs.randint(-2, 3, sh).astype(np.float32)
    else:
        f = lambda *sh: rs.standard_normal(sh).astype(np.float32)
    t = dict(x=f(N, C, H, W), w=(f(C, R, S) if ties else 0.3 * f(C, R, S)).astype(np.float32),
             w2=(f(C, R, S) if ties else 0.3 * f(C, R, S)).astype(np.float32),
             alpha=rs.uniform(-1, 1, C).astype(np.float32), beta=rs.uniform(-1, 1, C).astype(np.float32),
             bias=rs.uniform(-0.1, 0.1, C).astype(np.float32), g=f(N, C, OH, OW))
    if d["dtype"] == "bf16":
        for k in ("x", "w", "w2", "g"):
            t[k] = inputs.to_bf16_values(t[k])
    return t


def check(d, seed, ties=False, null_ab=False):
    t = draw(d, seed, ties)
    two, par = d["mode"] in ("compound", "parallel"), d["mode"] == "parallel"
    dt = tconv.TORCH_DTYPE[d["dtype"]]
    dev = lambda a, ty=None: torch.from_numpy(a).cuda().to(ty) if ty else torch.from_numpy(a).cuda()
    al = t["alpha"] if (two and not null_ab) else None
    be = t["beta"] if (two and not null_ab) else None
    ref = ora.depthwise_forward(d, t["x"], t["w"], t["w2"] if par else None, al, be, t["bias"])
    gx, gw, gw2 = dev(t["x"], dt), dev(t["w"], dt), dev(t["w2"], dt) if par else None
    ga, gb = (dev(al) if al is not None else None), (dev(be) if be is not None else None)
    y, win = tconv.dw_forward(d, gx, gw, gw2, ga, gb, dev(t["bias"]), want_winners=True)
    y0, _ = tconv.dw_forward(d, gx, gw, gw2, ga, gb, dev(t["bias"]), want_winners=False)
    torch.cuda.synchronize()
    want = inputs.to_bf16_values(ref["y"]) if d["dtype"] == "bf16" else ref["y"]
    for out in (y, y0):
        assert parity.same_bits(out.float().cpu().numpy(), want).all(), (d, tconv.tconv_last_kernel())
    assert np.array_equal(win.cpu().numpy(), ref["codes"]), d
    gref = ora.depthwise_backward(d, t["x"], t["w"], t["g"], t["w2"] if par else None, al, be)
    for winners in (win, None):       # stored codes, then recomputed into the workspace
        got = tconv.dw_backward(d, gx, gw, dev(t["g"], dt), gw2, ga, gb, winners)
        torch.cuda.synchronize()
        parity.compare_grads(d, got, gref)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("mode", MODES)
def test_depthwise_geometries(mode, dtype):
    mk = lambda N, C, H, W, R, S, **k: inputs.layer(N, C, H, W, C, R, S, mode=mode, dtype=dtype, **k)
    cases = [mk(2, 5, 9, 11, 3, 3, stride=1, pad=1),          # ragged width
             mk(3, 8, 16, 16, 3, 3, stride=2, pad=1),         # the stride-2 depthwise of an inverted residual
             mk(2, 5, 7, 7, 3, 3, stride=2, pad=1),           # stride 2 on odd extents (7 -> 4)
             mk(2, 3, 10, 13, 3, 3, stride=2, pad=1),         # stride 2, even height, odd width
             mk(2, 4, 12, 20, 3, 3, stride=1, pad=2, dil=2),
             mk(2, 3, 7, 7, 3, 3, stride=1, pad=0),           # no padding
             mk(1, 6, 10, 9, 1, 3, stride=1, pad=1),          # 1 x 3 window
             mk(2, 2, 9, 9, 4, 4, stride=1, pad=1),           # 16 taps: the most a code nibble holds
             mk(5, 3, 4, 4, 3, 3, stride=1, pad=1)]           # tiny planes
    for i, d in enumerate(cases):
        check(d, 3000 + i)
        check(d, 3100 + i, ties=True)


def test_depthwise_null_alpha_beta_and_mobilenet_shape():
    check(inputs.layer(2, 4, 8, 8, 4, 3, 3, pad=1, mode="compound"), 3200, null_ab=True)
    # a MobileNetV2 stage shape at reduced batch: 96 channels on 14 x 14... and 32 x 32 (CIFAR-sized input)
    check(inputs.layer(2, 96, 14, 14, 96, 3, 3, pad=1, mode="compound", dtype="bf16"), 3201)
    check(inputs.layer(2, 32, 32, 32, 32, 3, 3, pad=1, mode="parallel"), 3202)


def test_depthwise_descriptor_checks():
    d = inputs.layer(1, 4, 8, 8, 5, 3, 3, pad=1, mode="compound")           # K != C
    assert tconv.tconv_dw_winner_bytes(d) == 0
    x = torch.zeros(1, 4, 8, 8, device="cuda"); w = torch.zeros(4, 3, 3, device="cuda")
    y = torch.zeros(1, 5, 8, 8, device="cuda")
    assert tconv.tconv_dw_forward(d, x, w, None, None, None, None, y) == -1
    d = inputs.layer(1, 4, 9, 9, 4, 5, 5, pad=2, mode="compound")           # 25 taps
    assert tconv.tconv_dw_forward(d, x, w, None, None, None, None, y) == -2
    d = inputs.layer(1, 4, 8, 8, 4, 3, 3, pad=1, mode="parallel")           # parallel needs w2
    y = torch.zeros(1, 4, 8, 8, device="cuda")
    assert tconv.tconv_dw_forward(d, x, w, None, None, None, None, y) == -1


@pytest.mark.parametrize("dtype,N,stride", [("f32", 128, 1), ("bf16", 16, 1), ("f32", 32, 2), ("bf16", 8, 2)])
def test_depthwise_at_the_benchmark_size(dtype, N, stride):
    """The layer `bench.py --workload dw` times (144 channels, 56 x 56, 3 x 3, padding 1, compound) in
    full against the oracle, and its stride-2 form (the bf16 oracle is slower: fewer images)."""
    check(inputs.layer(N, 144, 56, 56, 144, 3, 3, stride=stride, pad=1, mode="compound", dtype=dtype), 3300 + N)
