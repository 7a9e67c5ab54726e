"""The any-shape kernels on the shapes the tiled kernels normally take (3 x 3 windows, several
tiles): TCONV_FORCE_GENERIC=1 routes every call to them (the switch is read once per process, so
the checks run in a child process), and forward, winners and gradients are compared with the
oracle as in the other parity tests."""
import os
import subprocess
import sys
from pathlib import Path

import pytest

pytestmark = pytest.mark.gpu
ROOT = Path(__file__).resolve().parent.parent

CHILD = r"""
import sys
sys.path.insert(0, %r); sys.path.insert(0, %r)
from paper_2504_06881_b200 import inputs, tconv
import parity
ALL = [("max_plus", "max"), ("min_plus", "min"), ("max_plus", "sum"), ("min_plus", "sum"), ("max_plus", "min"),
       ("min_plus", "max"), ("compound", "sum"), ("parallel", "sum")]
n = 0
for dtype in ("f32", "bf16"):
    for mode, chan in ALL:
        for geom in (dict(stride=1, pad=1), dict(stride=2, pad=1), dict(stride=1, pad=2, dil=2)):
            d = inputs.layer(2, 5, 20, 24, 9, 3, 3, mode=mode, chan=chan, dtype=dtype, **geom)
            parity.check_forward(d, inputs.draw(d, 900 + n))
            assert tconv.tconv_last_kernel() == "fwd_generic", tconv.tconv_last_kernel()
            parity.check_layer(d, None, 900 + n, recompute=(n %% 3 == 0))
            assert tconv.tconv_last_kernel() == "bwd_generic", tconv.tconv_last_kernel()
            parity.check_layer(d, dict(x=("ints", -1, 1), w=("ints", -1, 1)), 950 + n, recompute=False)
            n += 1
print("checked", n)
"""


def test_any_shape_kernels_on_tiled_shapes():
    env = dict(os.environ, TCONV_FORCE_GENERIC="1")
    out = subprocess.run([sys.executable, "-c", CHILD % (str(ROOT), str(ROOT / "tests"))], env=env,
                         capture_output=True, text=True, timeout=900)
    assert out.returncode == 0, out.stdout[-1500:] + out.stderr[-3000:]
    assert "checked 48" in out.stdout


CHILD_1D = r"""
import sys
sys.path.insert(0, %r); sys.path.insert(0, %r)
import torch
from paper_2504_06881_b200 import inputs, tconv3d
from test_gpu_3d import check
n = 0
for dtype in ("f32", "bf16"):
    for mode, chan in (("max_plus", "default"), ("min_plus", "sum"), ("compound", "default"), ("parallel", "default")):
        d = inputs.layer3d(2, 2, 1, 1, 600, 5, T=1, R=1, S=80, stride=(1, 1, 4), mode=mode, chan=chan, dtype=dtype)
        check(d, 980 + n)
        n += 1
# the any-shape backward of a compound layer takes eight launches, the one-dimensional one seven
d = inputs.layer3d(2, 1, 1, 1, 400, 8, T=1, R=1, S=80, stride=(1, 1, 4), mode="compound")
t = inputs.draw3d(d, 990)
dev = lambda a: torch.from_numpy(a).cuda()
y, win = tconv3d.forward(d, dev(t["x"]), dev(t["w"]), None, dev(t["alpha"]), dev(t["beta"]), dev(t["bias"]), want_winners=True)
l0 = tconv3d.tconv3d_launch_count()
tconv3d.backward(d, dev(t["x"]), dev(t["w"]), dev(t["g"]), None, dev(t["alpha"]), dev(t["beta"]), win)
assert tconv3d.tconv3d_launch_count() - l0 == 8
print("checked", n)
"""


def test_any_shape_kernels_on_one_dimensional_shapes():
    """Long 1-D windows through the any-shape kernels of the three-dimensional entry points (the
    path taken by dilated or oddly strided 1-D layers), against the oracle."""
    env = dict(os.environ, TCONV_FORCE_GENERIC="1")
    out = subprocess.run([sys.executable, "-c", CHILD_1D % (str(ROOT), str(ROOT / "tests"))], env=env,
                         capture_output=True, text=True, timeout=900)
    assert out.returncode == 0, out.stdout[-1500:] + out.stderr[-3000:]
    assert "checked 8" in out.stdout
