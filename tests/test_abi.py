"""The C-ABI library loads, exports every declared symbol, and its host-side checks work
(no compute call needs a GPU here)."""
import ctypes
import re
from pathlib import Path

import pytest

from paper_2504_06881_b200 import inputs, tconv

ROOT = Path(__file__).resolve().parent.parent


def test_every_declared_symbol_is_exported():
    from paper_2504_06881_b200 import tconv3d
    lib = ctypes.CDLL(str(tconv.LIB_PATH))
    headers = sorted((ROOT / "include").glob("*.h"))
    assert [h.name for h in headers] == ["tconv.h", "tconv3d.h"]
    for header, symbols in zip(headers, (tconv.SYMBOLS, tconv3d.SYMBOLS)):
        declared = set(re.findall(r"\b(tconv(?:3d)?_[a-z0-9_]+)\s*\(", header.read_text()))
        assert declared, "no declarations found"
        for name in declared:
            assert hasattr(lib, name), f"{name} declared in {header.name} but not exported"
        assert declared == set(symbols), header.name


def test_output_shape_and_sizes():
    d = inputs.layer(2, 3, 32, 32, 16, 3, 3, stride=1, pad=1, mode="compound")
    assert tconv.tconv_output_shape(d) == (32, 32)
    assert tconv.tconv_winner_bytes(d) == 2 * 16 * 3 * 32 * 32
    assert tconv.tconv_winner_bytes(dict(d, mode="max_plus")) == 4 * 2 * 16 * 32 * 32
    assert tconv.tconv_winner_bytes(dict(d, R=5, S=5)) == 2 * 2 * 16 * 3 * 30 * 32      # code rows padded to 4
    assert tconv.tconv_winner_bytes(dict(d, W=9)) == 2 * 16 * 3 * 32 * 12
    assert tconv.tconv_winner_bytes(dict(d, W=9, mode="max_plus")) == 4 * 2 * 16 * 32 * 9
    assert tconv.tconv_workspace_bytes(d, True) >= tconv.tconv_winner_bytes(d)
    d2 = inputs.layer(1, 1, 56, 56, 1, 3, 3, stride=2, pad=1, dil=1)
    assert tconv.tconv_output_shape(d2) == (28, 28)
    d3 = inputs.layer(1, 1, 128, 256, 1, 3, 3, stride=1, pad=2, dil=2)
    assert tconv.tconv_output_shape(d3) == (128, 256)


def test_paper_op_counts_match_section_4_1():
    N, C, H, W, K, R, S = 2, 5, 9, 8, 3, 3, 3
    P = N * K * 7 * 6
    d = inputs.layer(N, C, H, W, K, R, S)
    assert tconv.tconv_paper_ops(dict(d, mode="max_plus")) == (2 * R * S * C - 1) * P
    assert tconv.tconv_paper_ops(dict(d, mode="min_plus", chan="sum")) == \
        ((C - 1 + R * S * C) + (R * S - 1) * C) * P
    assert tconv.tconv_paper_ops(dict(d, mode="compound")) == \
        ((R * S * C + 2 * C - 1) + 2 * (R * S - 1) * C + 2 * C) * P
    assert tconv.tconv_paper_ops(dict(d, mode="parallel")) == \
        ((2 * R * S * C + 2 * C - 1) + 2 * (R * S - 1) * C + 2 * C) * P


def test_host_side_argument_checks():
    d = inputs.layer(1, 1, 4, 4, 1, 3, 3)
    with pytest.raises(tconv.TconvError):
        tconv.tconv_output_shape(dict(d, H=0))
    with pytest.raises(tconv.TconvError):
        tconv.tconv_output_shape(dict(d, H=2))          # window larger than the padded input
    with pytest.raises(tconv.TconvError) as e:
        tconv.tconv_output_shape(dict(d, mode="compound", chan="max"))
    assert e.value.status == -2
    assert tconv.tconv_winner_bytes(dict(d, stride_h=0)) == 0
    lib = ctypes.CDLL(str(tconv.LIB_PATH))
    lib.tconv_forward.restype = ctypes.c_int
    desc = tconv.make_desc(d)
    vp = ctypes.c_void_p
    args = [ctypes.byref(desc)] + [vp(0)] * 9 + [ctypes.c_size_t(0), vp(0)]
    assert lib.tconv_forward(*args) == -1                # NULL tensors
    args[1] = vp(0x1008); args[2] = vp(0x1000); args[7] = vp(0x1000)
    assert lib.tconv_forward(*args) == -3                # misaligned x
    assert tconv.tconv_status_string(-3).startswith("pointer")
    assert tconv.tconv_alu_probe_name(0) == "f32_add_max2"
    assert tconv.tconv_alu_probe_name(10_000) is None


def test_empty_and_oversized_descriptors_are_rejected_on_the_host():
    """Empty tensors (a zero extent) are invalid arguments; layers whose flat indices would not fit
    the launch arithmetic are refused with TCONV_ERR_TOO_LARGE before anything is launched."""
    d = inputs.layer(1, 1, 4, 4, 1, 3, 3, pad=1)
    for key in ("N", "C", "K", "H", "W", "R", "S"):
        with pytest.raises(tconv.TconvError) as e:
            tconv.tconv_output_shape(dict(d, **{key: 0}))
        assert e.value.status == -1
        assert tconv.tconv_winner_bytes(dict(d, **{key: 0})) == 0
        assert tconv.tconv_workspace_bytes(dict(d, **{key: 0}), True) == 0
    big = inputs.layer(2_000_000, 512, 1024, 1024, 512, 3, 3, pad=1)      # 1e15 outputs
    with pytest.raises(tconv.TconvError) as e:
        tconv.tconv_output_shape(big)
    assert e.value.status == -7
    assert tconv.tconv_status_string(-7) != ""
    with pytest.raises(tconv.TconvError) as e:                             # more than 256 taps
        tconv.tconv_output_shape(inputs.layer(1, 1, 40, 40, 1, 17, 17))
    assert e.value.status == -2


def test_depthwise_descriptor_checks_on_the_host():
    ok = inputs.layer(2, 8, 9, 9, 8, 3, 3, pad=1, mode="compound")
    assert tconv.tconv_dw_winner_bytes(ok) == 2 * 8 * 9 * 9
    assert tconv.tconv_dw_workspace_bytes(ok, False) == 0
    assert tconv.tconv_dw_workspace_bytes(ok, True) >= tconv.tconv_dw_winner_bytes(ok)
    assert tconv.tconv_dw_winner_bytes(dict(ok, K=4)) == 0                 # one output channel per input channel
    assert tconv.tconv_dw_winner_bytes(dict(ok, R=5, S=5, pad_h=2, pad_w=2)) == 0   # a code nibble holds 16 taps
    assert tconv.tconv_dw_winner_bytes(dict(ok, N=0)) == 0
    assert tconv.tconv_dw_winner_bytes(inputs.layer(70_000, 1024, 64, 64, 1024, 3, 3, pad=1)) == 0   # > 2^31 - 1 elements


def test_three_dimensional_descriptor_checks():
    """Host-side calls of include/tconv3d.h (no GPU needed)."""
    from paper_2504_06881_b200 import tconv3d
    d = inputs.layer3d(1, 1, 4, 4, 4, 1, T=3, R=3, S=3)
    assert tconv3d.tconv3d_output_shape(d) == (2, 2, 2)
    assert tconv3d.tconv3d_output_shape(inputs.layer3d(2, 1, 28, 28, 28, 6, T=5, R=5, S=5, stride=2)) == (12, 12, 12)
    assert tconv3d.tconv3d_output_shape(dict(d, D=9, H=8, W=7, stride=(2, 1, 3), pad=(1, 0, 2), dil=(2, 1, 1))) == (4, 6, 3)
    assert tconv3d.tconv3d_winner_bytes(d) == 4 * 8                     # int32 per output
    assert tconv3d.tconv3d_winner_bytes(dict(d, chan="sum")) == 2 * 8   # uint16 per (output, channel)
    assert tconv3d.tconv3d_winner_bytes(dict(d, C=3, mode="compound")) == 2 * 3 * 8
    assert tconv3d.tconv3d_winner_bytes(dict(d, T=9, R=9, S=9, pad=(4, 4, 4))) == 0      # > 256 taps
    assert tconv3d.tconv3d_workspace_bytes(d, False) == 0
    assert tconv3d.tconv3d_workspace_bytes(d, True) >= tconv3d.tconv3d_winner_bytes(d)
    with pytest.raises(tconv.TconvError):
        tconv3d.tconv3d_output_shape(dict(d, D=2))                       # window larger than the volume
    with pytest.raises(tconv.TconvError) as e:
        tconv3d.tconv3d_output_shape(dict(d, mode="compound", chan="max"))
    assert e.value.status == -2
    for key in ("N", "C", "D", "H", "W", "K", "T", "R", "S"):
        assert tconv3d.tconv3d_winner_bytes(dict(d, **{key: 0})) == 0
    assert tconv3d.tconv3d_winner_bytes(dict(d, stride=(0, 1, 1))) == 0
    assert tconv3d.tconv3d_winner_bytes(inputs.layer3d(4096, 64, 64, 64, 64, 64, pad=1)) == 0   # > 2^31 - 1 elements
