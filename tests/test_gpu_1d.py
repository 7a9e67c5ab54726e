"""Parity of the one-dimensional kernels (long windows through the three-dimensional entry points:
unit depth and height, 1 x 1 x S window) with the three-dimensional oracle: forward outputs and
winners bit for bit, gradients within the tolerance of the dense layers.  Shapes: the opening layer
of the paper's audio networks (one input channel, window 80, stride 4) on a shortened signal,
every stride the kernels take, windows that are no multiple of the stride, padding, ragged tiles of
positions and of output channels, several input channels, ties."""
import pytest

from paper_2504_06881_b200 import inputs
from test_gpu_3d import MODES, check

pytestmark = pytest.mark.gpu


def layer1d(N, C, L, K, S, stride=1, pad=0, **kw):
    return inputs.layer3d(N, C, 1, 1, L, K, T=1, R=1, S=S, stride=(1, 1, stride), pad=(0, 0, pad), **kw)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("mode,chan", MODES)
def test_audio_opening_layer(mode, chan, dtype):
    """Window 80, stride 4, one input channel; 1900 samples give 456 positions: three full tiles of
    128 and a ragged one; 36 output channels leave a ragged group."""
    check(layer1d(3, 1, 1900, 36, 80, stride=4, mode=mode, chan=chan, dtype=dtype), 1101)


@pytest.mark.parametrize("mode,chan", [("max_plus", "default"), ("min_plus", "sum"), ("compound", "default"),
                                       ("parallel", "default")])
@pytest.mark.parametrize("S,stride,pad", [(4, 1, 0), (7, 1, 3), (9, 2, 4), (33, 2, 0), (16, 4, 8), (81, 4, 40),
                                          (256, 1, 17), (255, 4, 0), (5, 4, 2)])
def test_windows_strides_and_padding(mode, chan, S, stride, pad):
    check(layer1d(2, 3, 700, 5, S, stride=stride, pad=pad, mode=mode, chan=chan), 1102 + S)


@pytest.mark.parametrize("mode,chan", MODES)
def test_integer_inputs_with_ties(mode, chan):
    d = layer1d(2, 4, 300, 9, 12, stride=2, pad=3, mode=mode, chan=chan)
    check(d, 1103, dists=dict(x=("ints", -1, 1), w=("ints", -1, 1)))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_many_channels_and_parameter_free(dtype):
    check(layer1d(2, 17, 513, 40, 10, stride=2, mode="compound", dtype=dtype), 1104, null_ab=True, use_bias=False)
    check(layer1d(1, 8, 260, 33, 31, stride=1, pad=15, mode="parallel", dtype=dtype), 1105)


def test_signal_shorter_than_a_tile_and_single_position():
    check(layer1d(2, 2, 80, 3, 80, stride=4, mode="compound"), 1106)
    check(layer1d(1, 1, 95, 130, 80, stride=4, mode="max_plus"), 1107)


def test_runs_on_the_one_dimensional_kernels():
    """The fast path is the one these tests exercise: its launch count differs from the any-shape
    path's (forward 1 launch either way; backward of a compound layer 7 against 8)."""
    import torch
    from paper_2504_06881_b200 import tconv, tconv3d
    d = layer1d(2, 1, 400, 8, 80, stride=4, mode="compound")
    t = inputs.draw3d(d, 1108)
    dev = lambda a: torch.from_numpy(a).cuda()
    y, win = tconv3d.forward(d, dev(t["x"]), dev(t["w"]), None, dev(t["alpha"]), dev(t["beta"]), dev(t["bias"]),
                             want_winners=True)
    l0 = tconv3d.tconv3d_launch_count()
    tconv3d.backward(d, dev(t["x"]), dev(t["w"]), dev(t["g"]), None, dev(t["alpha"]), dev(t["beta"]), win)
    torch.cuda.synchronize()
    assert tconv3d.tconv3d_launch_count() - l0 == 7


@pytest.mark.parametrize("seed", [1201, 1202, 1203])
def test_seeded_random_one_dimensional_layers(seed):
    """Twelve random layers per seed: window 4..256, stride 1, 2, 4 (the 1-D kernels) or 3 (any-shape
    kernels), padding up to half the window, 1..6 input and 1..40 output channels, both dtypes, every
    mode and channel combine."""
    import numpy as np
    rs = np.random.RandomState(seed)
    done = 0
    while done < 12:
        mode, chan = MODES[rs.randint(len(MODES))]
        S = int(rs.choice([4, 5, 7, 12, 16, 31, 64, 80, 100, 129, 256]))
        st = int(rs.choice([1, 2, 4, 4, 3]))
        L = int(rs.randint(S, 4 * S + 300))
        d = layer1d(int(rs.randint(1, 4)), int(rs.randint(1, 7)), L, int(rs.randint(1, 41)), S, stride=st,
                    pad=int(rs.randint(0, S // 2 + 1)), mode=mode, chan=chan, dtype=["f32", "bf16"][rs.randint(2)])
        if min(inputs.output_dhw(d)) <= 0:
            continue
        done += 1
        ties = rs.rand() < 0.3
        check(d, seed * 100 + done, dists=dict(x=("ints", -2, 2), w=("ints", -1, 1)) if ties else None)


@pytest.mark.parametrize("mode,dtype,N", [("compound", "f32", 32), ("max_plus", "f32", 32), ("parallel", "bf16", 4)])
def test_audio_opening_layer_at_the_benchmark_size(mode, dtype, N):
    """The layer `bench.py --workload conv1d` times (32 signals of 16000 samples, 128 output channels,
    window 80, stride 4), in full against the oracle: forward, winners and every gradient (the bf16
    oracle is slower: four signals)."""
    check(layer1d(N, 1, 16000, 128, 80, stride=4, mode=mode, dtype=dtype), 1300)
