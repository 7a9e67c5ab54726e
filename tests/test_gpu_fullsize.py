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


def full_size_check(d, dist, seed, sample_n, sample_k):
    return parity.sampled_check(d, inputs.draw(d, seed, **dist), sample_n, sample_k)


@pytest.mark.parametrize("mode", ["max_plus", "min_plus", "compound", "parallel"])
def test_cfg2_full_size(mode):
    """N=128, C=K=64, 32x32, fp32: the step bench.py times."""
    d, dist = inputs.cfg2(mode)
    k = full_size_check(d, dist, 1020, sample_n=(0, 77, 127), sample_k=(24, 40))
    assert "tma" in k


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_cfg3a_full_size(dtype):
    """ImageNet-scale mid layer, parallel, N=64, C=K=128, 28x28."""
    d, dist = inputs.cfg3a(dtype)
    full_size_check(d, dist, 1030, sample_n=(5, 63), sample_k=(120, 128))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_cfg3b_full_size(dtype):
    """Stride-2 variant, C=64 -> K=128 from 56x56."""
    d, dist = inputs.cfg3b(dtype)
    full_size_check(d, dist, 1031, sample_n=(0, 31), sample_k=(0, 8))


def test_cfg4_full_size():
    """Segmentation-scale map, compound bf16, N=8, C=K=256, 128x256, dilation 2."""
    d, dist = inputs.cfg4("bf16")
    k = full_size_check(d, dist, 1040, sample_n=(7,), sample_k=(100, 102))
    assert "bf16_tma" in k
