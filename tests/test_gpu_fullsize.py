"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

The oracle cannot run a whole full-size layer in seconds, so it computes a sample one piece
at a time: a few images x a slice of output channels.  The forward outputs and winners of
that sample are compared bit for bit with the full-size GPU run.  For the backward pass the
upstream gradient is zeroed outside the sample; then grad_x of the sampled images and the
parameter gradients of the sampled output channels equal what the oracle computes on the
sliced problem, and every other gradient element must be exactly zero.
"""
import numpy as np
import pytest
import torch

from oracle import tconv_oracle as ora
from paper_2504_06881_b200 import inputs, tconv
import parity

pytestmark = pytest.mark.gpu


def full_size_check(d, dist, seed, sample_n, sample_k, **more):
    return parity.sampled_check(d, inputs.draw(d, seed, **dist), sample_n, sample_k, **more)


# every (mode, channel combine) pair the benchmark tables list at this size
CFG2_CASES = [("max_plus", "default"), ("min_plus", "default"), ("compound", "default"), ("parallel", "default"),
              ("max_plus", "sum"), ("min_plus", "sum"), ("max_plus", "min"), ("min_plus", "max")]


@pytest.mark.parametrize("mode,chan", CFG2_CASES)
def test_cfg2_full_size(mode, chan):
    """N=128, C=K=64, 32x32, fp32: the step bench.py times.  Forward, winners and backward on
    three images x 16 output channels that straddle two k-tiles; forward and winners of the
    last image over every output channel and of 1024 random outputs."""
    d, dist = inputs.cfg2(mode, chan)
    k = full_size_check(d, dist, 1020, sample_n=(0, 77, 127), sample_k=(24, 40),
                        fwd_blocks=[(127, 0, 64)], random_outputs=1024, random_seed=1021)
    assert "tma" in k


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_cfg3a_full_size(dtype):
    """ImageNet-scale mid layer, parallel, N=64, C=K=128, 28x28: 32 output channels across a
    k-tile boundary, forward of the first image over all channels, 2048 random outputs."""
    d, dist = inputs.cfg3a(dtype)
    full_size_check(d, dist, 1030, sample_n=(5, 63), sample_k=(80, 112),
                    fwd_blocks=[(0, 0, 128)], random_outputs=2048, random_seed=1032)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_cfg3b_full_size(dtype):
    """Stride-2 variant, C=64 -> K=128 from 56x56."""
    d, dist = inputs.cfg3b(dtype)
    full_size_check(d, dist, 1031, sample_n=(0, 31), sample_k=(16, 48),
                    fwd_blocks=[(63, 0, 128)], random_outputs=2048, random_seed=1033)


def test_cfg4_full_size():
    """Segmentation-scale map, compound bf16, N=8, C=K=256, 128x256, dilation 2: forward and
    winners of image 0 over all 256 output channels and of 4096 random outputs of the other
    images; backward on image 0 for the 32 output channels 112..143 (two k-tiles), the upstream
    gradient zero elsewhere; forward of the last image on the first and the last k-tile."""
    d, dist = inputs.cfg4("bf16")
    k = full_size_check(d, dist, 1040, sample_n=(0,), sample_k=(112, 144),
                        fwd_blocks=[(0, 0, 112), (0, 144, 256), (7, 0, 32), (7, 224, 256)],
                        random_outputs=4096, random_seed=1041)
    assert "bf16_tma" in k
