"""Seeded random layer descriptors against the oracle: every mode, channel combine and dtype,
3x3 and other windows, strides and dilations 1-3, arbitrary and 'same' padding, widths that do and
do not divide into quads / 16-byte rows; dense and depthwise forms; random and tie-heavy inputs;
stored and recomputed winners.  Forward and winners bit for bit, gradients within tolerance."""
import numpy as np
import pytest

from paper_2504_06881_b200 import inputs, tconv
import parity
import test_gpu_depthwise as tdw

pytestmark = pytest.mark.gpu

ALL = [("max_plus", "max"), ("max_plus", "sum"), ("max_plus", "min"), ("min_plus", "min"), ("min_plus", "sum"),
       ("min_plus", "max"), ("compound", "sum"), ("parallel", "sum")]
WINDOWS = [(3, 3), (3, 3), (3, 3), (3, 3), (1, 1), (1, 3), (3, 1), (2, 2), (5, 5), (4, 4)]


@pytest.mark.parametrize("seed", [11, 12, 13, 14])
def test_random_descriptors(seed):
    rs = np.random.RandomState(seed)
    done = 0
    while done < 60:
        mode, chan = ALL[rs.randint(len(ALL))]
        dtype = ["f32", "bf16"][rs.randint(2)]
        R, S = WINDOWS[rs.randint(len(WINDOWS))]
        st, dl = [1, 1, 1, 2, 2, 3][rs.randint(6)], [1, 1, 1, 2, 2, 3, 4, 4][rs.randint(8)]
        pad = rs.randint(0, 3) if rs.rand() < 0.5 else (S - 1) * dl // 2
        N, C, K = rs.randint(1, 12), rs.randint(1, 60), rs.randint(1, 80)
        H = rs.randint(1, 48)
        W = [rs.randint(1, 70), 4 * rs.randint(1, 16), 8 * rs.randint(1, 8), 28, 14, 7][rs.randint(6)]
        d = inputs.layer(N, C, H, W, K, R, S, stride=st, pad=pad, dil=dl, mode=mode, chan=chan, dtype=dtype)
        if min(inputs.output_hw(d)) <= 0:
            continue
        OH, OW = inputs.output_hw(d)
        if N * K * C * R * S * OH * OW > 1.5e8:
            continue
        dist = None if rs.rand() < 0.6 else dict(x=("ints", -2, 2), w=("ints", -2, 2))
        parity.check_layer(d, dist, int(rs.randint(1 << 30)), recompute=bool(rs.randint(2)))
        assert tconv.tconv_device_status() == 0
        if rs.rand() < 0.4 and R * S <= 16:
            dd = inputs.layer(N, C, H, W, C, R, S, stride=st, pad=pad, dil=dl, mode=mode, dtype=dtype)
            tdw.check(dd, int(rs.randint(1 << 30)), ties=bool(rs.randint(2)))
        done += 1


@pytest.mark.parametrize("seed", [21, 22])
def test_random_three_dimensional_descriptors(seed):
    import test_gpu_3d as t3
    rs = np.random.RandomState(seed)
    done = 0
    while done < 40:
        mode, chan = ALL[rs.randint(len(ALL))]
        dtype = ["f32", "bf16"][rs.randint(2)]
        T, R, S = (int(rs.randint(1, 6)) for _ in range(3))
        stride = tuple(int(v) for v in rs.randint(1, 4, 3))
        dil = tuple(int(v) for v in rs.randint(1, 3, 3))
        pad = tuple(int(v) for v in rs.randint(0, 3, 3))
        N, C, K = int(rs.randint(1, 5)), int(rs.randint(1, 20)), int(rs.randint(1, 20))
        D, H, W = (int(rs.randint(1, 20)) for _ in range(3))
        d = inputs.layer3d(N, C, D, H, W, K, T=T, R=R, S=S, stride=stride, pad=pad, dil=dil, mode=mode,
                           chan=chan, dtype=dtype)
        od = inputs.output_dhw(d)
        if min(od) <= 0 or N * K * C * T * R * S * od[0] * od[1] * od[2] > 3e7:
            continue
        dist = None if rs.rand() < 0.6 else dict(x=("ints", -2, 2), w=("ints", -2, 2))
        t3.check(d, int(rs.randint(1 << 30)), dists=dist)
        done += 1
