"""Failure detection without a GPU fault: a bounded wait of the copy-engine kernels is made to run
out (a test-only environment switch makes the kernel skip the copies of its first chunk, so nothing
is in flight, and sets the poll limit), and the host sees TCONV_ERR_DEVICE_TIMEOUT once, then a
clean status; the context stays usable.  Runs in child processes because the switch is read once
per process."""
import json
import os
import subprocess
import sys
from pathlib import Path

import pytest

pytestmark = pytest.mark.gpu
ROOT = Path(__file__).resolve().parent.parent

CHILD = r"""
import json, sys, time, torch
sys.path.insert(0, %r)
from paper_2504_06881_b200 import inputs, tconv
d = inputs.layer(1, 16, 4, 32, 16, 3, 3, stride=1, pad=1, mode="compound")       # one CTA
x = torch.randn(1, 16, 4, 32, device="cuda"); w = torch.randn(16, 16, 3, 3, device="cuda")
torch.cuda.synchronize()
t0 = time.perf_counter()
y, _ = tconv.forward(d, x, w)
kernel = tconv.tconv_last_kernel()
torch.cuda.synchronize()
dt = time.perf_counter() - t0
first = tconv.tconv_device_status()
second = tconv.tconv_device_status()
# the context is still usable: a plain torch kernel runs and gives the right answer
ok = bool((torch.arange(8, device="cuda").sum() == 28).item())
print(json.dumps({"kernel": kernel, "seconds": dt, "first": first, "second": second, "usable": ok}))
"""


def _run(switch):
    env = dict(os.environ, TCONV_DEBUG_DROP_COPY=str(switch))
    out = subprocess.run([sys.executable, "-c", CHILD % str(ROOT)], env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    return json.loads(out.stdout.strip().splitlines()[-1])


def test_bounded_wait_runs_out_and_reports_a_timeout():
    """The kernel waits twice on the dropped chunk (2^16 polls each, measured 4 us per poll) and
    returns: the give-up takes about half a second, the host reads the timeout once."""
    r = _run(1)
    assert "tma" in r["kernel"]
    assert r["first"] == -6 and r["second"] == 0 and r["usable"]
    print("give-up time:", r["seconds"], "s")
    assert r["seconds"] < 5.0


def test_switch_off_leaves_the_layer_alone():
    r = _run(0)
    assert r["first"] == 0 and r["second"] == 0
