"""The paper's layer names over ``TropicalConv2d`` (layers (i)-(vi) of the section "Tropical algebra
and tropical convolution", the sections "Compound tropical convolution layers" and "Parallel
tropical convolution layers", appendix "Compatibility with PyTorch"): every class takes
``nn.Conv2d``'s constructor arguments.

Base operator + channel combine, in the paper's numbering:  MinPlusSumConv2d (i), MaxPlusSumConv2d
(ii), MinPlusMaxConv2d (iii), MinPlusMinConv2d (iv), MaxPlusMaxConv2d (v), MaxPlusMinConv2d (vi).
Compound / parallel with 0, 1 (beta = 1 - alpha) or 2 learnable scalar sets per (c_out, c_in).
"""
from __future__ import annotations

from .nn import TropicalConv2d


def _named(name, mode, chan="default", params="2p", doc="", base=TropicalConv2d):
    def __init__(self, in_channels, out_channels, kernel_size, stride=1, padding=0, dilation=1,
                 bias=True, dtype="f32", **kw):
        base.__init__(self, in_channels, out_channels, kernel_size, stride=stride,
                      padding=padding, dilation=dilation, bias=bias, mode=mode, chan=chan,
                      params=kw.pop("params", params), dtype=dtype, **kw)
    return type(name, (base,), {"__init__": __init__, "__doc__": doc})


MaxPlusSumConv2d = _named("MaxPlusSumConv2d", "max_plus", "sum", doc="layer (ii): sum over channels of the max-plus window")
MinPlusSumConv2d = _named("MinPlusSumConv2d", "min_plus", "sum", doc="layer (i): sum over channels of the min-plus window")
MinPlusMaxConv2d = _named("MinPlusMaxConv2d", "min_plus", "max", doc="layer (iii): max over channels of the min-plus window")
MinPlusMinConv2d = _named("MinPlusMinConv2d", "min_plus", "min", doc="layer (iv): min over channels and window")
MaxPlusMaxConv2d = _named("MaxPlusMaxConv2d", "max_plus", "max", doc="layer (v): max over channels and window")
MaxPlusMinConv2d = _named("MaxPlusMinConv2d", "max_plus", "min", doc="layer (vi): min over channels of the max-plus window")

CompoundMinMaxPlusSumConv2d0p = _named("CompoundMinMaxPlusSumConv2d0p", "compound", params="0p", doc="compound mode, alpha = beta = 1")
CompoundMinMaxPlusSumConv2d1p = _named("CompoundMinMaxPlusSumConv2d1p", "compound", params="1p", doc="compound mode, beta = 1 - alpha")
CompoundMinMaxPlusSumConv2d2p = _named("CompoundMinMaxPlusSumConv2d2p", "compound", params="2p", doc="compound mode, learnable alpha and beta")
ParallelMinMaxPlusSumConv2d0p = _named("ParallelMinMaxPlusSumConv2d0p", "parallel", params="0p", doc="parallel mode, alpha = beta = 1")
ParallelMinMaxPlusSumConv2d1p = _named("ParallelMinMaxPlusSumConv2d1p", "parallel", params="1p", doc="parallel mode, beta = 1 - alpha")
ParallelMinMaxPlusSumConv2d2p = _named("ParallelMinMaxPlusSumConv2d2p", "parallel", params="2p", doc="parallel mode, learnable alpha and beta")

__all__ = [n for n in dir() if n.endswith(("Conv2d", "0p", "1p", "2p"))]

from .nn import TropicalConv1d, TropicalConv3d, TropicalDepthwiseConv2d  # noqa: E402  (1-D, 3-D and depthwise forms)

# the three-dimensional layers of Section 3.2 and the Conv3d forms of Sections 3.4 / 3.5: the same
# names with Conv3d, ``nn.Conv3d``'s constructor arguments
_SPECS = {"MaxPlusSum": ("max_plus", "sum", "2p"), "MinPlusSum": ("min_plus", "sum", "2p"),
          "MinPlusMax": ("min_plus", "max", "2p"), "MinPlusMin": ("min_plus", "min", "2p"),
          "MaxPlusMax": ("max_plus", "max", "2p"), "MaxPlusMin": ("max_plus", "min", "2p")}
for _stem, (_mode, _chan, _params) in _SPECS.items():
    globals()[_stem + "Conv3d"] = _named(_stem + "Conv3d", _mode, _chan, doc=f"{_stem}Conv2d in three dimensions",
                                         base=TropicalConv3d)
    __all__.append(_stem + "Conv3d")
for _mode in ("compound", "parallel"):
    for _params in ("0p", "1p", "2p"):
        _name = f"{_mode.capitalize()}MinMaxPlusSumConv3d{_params}"
        globals()[_name] = _named(_name, _mode, params=_params, doc=f"{_mode} mode in three dimensions, {_params}",
                                  base=TropicalConv3d)
        __all__.append(_name)

__all__ += ["TropicalDepthwiseConv2d", "TropicalConv1d", "TropicalConv3d"]
