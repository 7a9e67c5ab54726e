"""PyTorch glue over the C ABI: an autograd Function, a drop-in layer and the
ResNet-18-shaped hybrid network of benchmark configuration 5.

Everything tropical runs in the library's CUDA kernels (forward with winners, winner-routed
backward); PyTorch supplies BatchNorm, the standard convolutions of the stem / stage 1 /
1x1 downsamples, the loss and the optimiser, none of which is on the tropical hot path.
The layer follows the paper's usage (Appendix "Compatibility with PyTorch"): same constructor
arguments as ``nn.Conv2d``; ``mode`` selects max_plus / min_plus / compound / parallel.
"""
from __future__ import annotations

import math

import torch
import torch.nn as nn

from . import tconv


class TropicalConvFn(torch.autograd.Function):
    """y = tconv_forward(x, w, w2, alpha, beta, bias); backward = tconv_backward with the stored winners.

    Master parameters may be fp32 while the layer computes in bf16: the cast happens here and the
    parameter gradients come back in fp32.  When ``TropicalConvFn.events`` is a list, every library
    call is bracketed by a pair of CUDA events appended to it (for the benchmark's per-layer times)."""

    events = None
    # True: bf16 layers read a float x directly (x_dtype) instead of a converted copy.  Off by default:
    # the conversion while staging rules out the copy-engine path, which costs more than the cast
    # kernel saves on the ResNet-18 shape (tropical forward 21.5 -> 23.9 ms per step).
    fuse_cast = False

    @staticmethod
    def forward(ctx, x, w, w2, alpha, beta, bias, geom):
        mode, chan, dtype, stride, pad, dil = geom
        dt = tconv.TORCH_DTYPE[dtype]
        N, C, H, W = x.shape
        K, _, R, S = w.shape
        d = dict(N=N, C=C, H=H, W=W, K=K, R=R, S=S, stride_h=stride[0], stride_w=stride[1],
                 pad_h=pad[0], pad_w=pad[1], dil_h=dil[0], dil_w=dil[1], mode=mode, chan=chan, dtype=dtype)
        # a float x for a bf16 layer is rounded by the kernel while it stages x (no cast kernel, no
        # bf16 copy); layers the tiled kernels do not serve fall back to the explicit cast
        fused_cast = TropicalConvFn.fuse_cast and dtype == "bf16" and x.dtype == torch.float32
        xc = x.detach().contiguous() if fused_cast else x.detach().to(dt).contiguous()
        if fused_cast:
            d["x_dtype"] = "f32"
        wc = w.detach().to(dt).contiguous()
        w2c = w2.detach().to(dt).contiguous() if w2 is not None else None
        al = alpha.detach().float().contiguous() if alpha is not None else None
        be = beta.detach().float().contiguous() if beta is not None else None
        bi = bias.detach().float().contiguous() if bias is not None else None
        need_grad = any(t is not None and t.requires_grad for t in (x, w, w2, alpha, beta, bias))
        ev = TropicalConvFn.events
        if ev is not None:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
        try:
            y, winners = tconv.forward(d, xc, wc, w2c, al, be, bi, want_winners=need_grad)
        except tconv.TconvError as err:
            if not fused_cast or err.status != -2:
                raise
            d.pop("x_dtype")
            xc = x.detach().to(dt).contiguous()
            y, winners = tconv.forward(d, xc, wc, w2c, al, be, bi, want_winners=need_grad)
        if ev is not None:
            e1.record()
            ev.append(("fwd", d, e0, e1))
        ctx.d = d
        ctx.in_dtype = x.dtype
        ctx.save_for_backward(xc, wc, w2c, al, be, winners)
        ctx.has = (w2 is not None, alpha is not None, beta is not None, bias is not None)
        return y.to(x.dtype) if x.dtype != dt else y

    @staticmethod
    def backward(ctx, gy):
        xc, wc, w2c, al, be, winners = ctx.saved_tensors
        d = ctx.d
        dt = tconv.TORCH_DTYPE[d["dtype"]]
        g = gy.to(dt).contiguous()
        ev = TropicalConvFn.events
        if ev is not None:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
        need = ["grad_w", "grad_w2", "grad_alpha", "grad_beta", "grad_bias"]
        if ctx.needs_input_grad[0]:
            need.append("grad_x")          # a first layer's input needs none: the kernel is skipped
        try:
            grads = tconv.backward(d, xc, wc, g, w2c, al, be, winners, need=tuple(need))
        except tconv.TconvError as err:
            if d.get("x_dtype") != "f32" or err.status != -2:
                raise
            d = {k: v for k, v in d.items() if k != "x_dtype"}      # a path that reads x itself: convert first
            grads = tconv.backward(d, xc.to(dt), wc, g, w2c, al, be, winners, need=tuple(need))
        if ev is not None:
            e1.record()
            ev.append(("bwd", d, e0, e1))
        has_w2, has_a, has_b, has_bias = ctx.has
        gx = grads["grad_x"].to(ctx.in_dtype) if "grad_x" in grads else None
        return (gx, grads["grad_w"], grads.get("grad_w2") if has_w2 else None,
                grads.get("grad_alpha") if has_a else None, grads.get("grad_beta") if has_b else None,
                grads["grad_bias"] if has_bias else None, None)


class TropicalConvBNFn(torch.autograd.Function):
    """Tropical layer followed by training-mode batch normalisation, the pair the paper's residual
    blocks are made of (section "ResNet Models").  The layer's kernel leaves the per-channel sums of
    y and y^2 (tconv_forward_stats), so the normalisation reads y once (scale and shift) instead of
    twice (statistics, then scale and shift).  Backward: the usual batch-normalisation gradient
    (channel reductions of grad and grad * y, then one elementwise pass), then tconv_backward."""

    @staticmethod
    def forward(ctx, x, w, w2, alpha, beta, gamma, bn_bias, geom, eps):
        mode, chan, dtype, stride, pad, dil = geom
        dt = tconv.TORCH_DTYPE[dtype]
        N, C, H, W = x.shape
        K, _, R, S = w.shape
        d = dict(N=N, C=C, H=H, W=W, K=K, R=R, S=S, stride_h=stride[0], stride_w=stride[1],
                 pad_h=pad[0], pad_w=pad[1], dil_h=dil[0], dil_w=dil[1], mode=mode, chan=chan, dtype=dtype)
        fused_cast = TropicalConvFn.fuse_cast and dtype == "bf16" and x.dtype == torch.float32
        xc = x.detach().contiguous() if fused_cast else x.detach().to(dt).contiguous()
        if fused_cast:
            d["x_dtype"] = "f32"
        wc = w.detach().to(dt).contiguous()
        w2c = w2.detach().to(dt).contiguous() if w2 is not None else None
        al = alpha.detach().float().contiguous() if alpha is not None else None
        be = beta.detach().float().contiguous() if beta is not None else None
        ev = TropicalConvFn.events
        if ev is not None:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
        try:
            y, winners, s1, s2 = tconv.forward_stats(d, xc, wc, w2c, al, be, None, want_winners=True)
        except tconv.TconvError as err:
            if not fused_cast or err.status != -2:
                raise
            d.pop("x_dtype")
            xc = x.detach().to(dt).contiguous()
            y, winners, s1, s2 = tconv.forward_stats(d, xc, wc, w2c, al, be, None, want_winners=True)
        if ev is not None:
            e1.record()
            ev.append(("fwd", d, e0, e1))
        cnt = float(y.shape[0] * y.shape[2] * y.shape[3])
        mean = s1 / cnt
        var = (s2 / cnt - mean * mean).clamp_min_(0.0)          # biased variance of the batch
        invstd = torch.rsqrt(var + eps)
        scale = gamma.detach().float() * invstd
        shift = bn_bias.detach().float() - mean * scale
        out = torch.addcmul(shift.view(1, -1, 1, 1), y, scale.view(1, -1, 1, 1))    # one pass over y, fp32 result
        ctx.d, ctx.in_dtype, ctx.cnt = d, x.dtype, cnt
        ctx.save_for_backward(xc, wc, w2c, al, be, winners, y, mean, invstd, gamma.detach().float())
        ctx.has = (w2 is not None, alpha is not None, beta is not None)
        ctx.mark_non_differentiable(mean, var)
        return out.to(x.dtype), mean, var

    @staticmethod
    def backward(ctx, go, _gm, _gv):
        xc, wc, w2c, al, be, winners, y, mean, invstd, gamma = ctx.saved_tensors
        d, cnt = ctx.d, ctx.cnt
        dt = tconv.TORCH_DTYPE[d["dtype"]]
        go = go.float()
        yf = y.float()
        sum_go = go.sum(dim=(0, 2, 3))
        sum_go_y = (go * yf).sum(dim=(0, 2, 3))
        sum_go_xmu = sum_go_y - mean * sum_go
        g_gamma = sum_go_xmu * invstd
        g_bias = sum_go
        # dy = gamma * invstd * (go - sum_go / cnt - (y - mean) * invstd^2 * sum_go_xmu / cnt)
        k1 = (gamma * invstd).view(1, -1, 1, 1)
        k2 = (invstd * invstd * sum_go_xmu / cnt).view(1, -1, 1, 1)
        k3 = (sum_go / cnt - mean * invstd * invstd * sum_go_xmu / cnt).view(1, -1, 1, 1)
        gy = (k1 * (go - yf * k2 - k3)).to(dt).contiguous()
        ev = TropicalConvFn.events
        if ev is not None:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
        need = ["grad_w", "grad_w2", "grad_alpha", "grad_beta"]
        if ctx.needs_input_grad[0]:
            need.append("grad_x")
        try:
            grads = tconv.backward(d, xc, wc, gy, w2c, al, be, winners, need=tuple(need))
        except tconv.TconvError as err:
            if d.get("x_dtype") != "f32" or err.status != -2:
                raise
            d = {k: v for k, v in d.items() if k != "x_dtype"}
            grads = tconv.backward(d, xc.to(dt), wc, gy, w2c, al, be, winners, need=tuple(need))
        if ev is not None:
            e1.record()
            ev.append(("bwd", d, e0, e1))
        has_w2, has_a, has_b = ctx.has
        gx = grads["grad_x"].to(ctx.in_dtype) if "grad_x" in grads else None
        return (gx, grads["grad_w"], grads.get("grad_w2") if has_w2 else None,
                grads.get("grad_alpha") if has_a else None, grads.get("grad_beta") if has_b else None,
                g_gamma, g_bias, None, None)


def tropical_conv_bn(conv: "TropicalConv2d", bn: nn.BatchNorm2d, x):
    """conv followed by bn; in training mode with the layer's fused channel statistics."""
    if not (bn.training and x.is_cuda and conv.bias is None and bn.affine and bn.track_running_stats
            and conv.params in ("2p", "0p") and type(conv) is TropicalConv2d):
        return bn(conv(x))
    geom = (conv.mode, conv.chan, conv.dtype, conv.stride, conv.padding, conv.dilation)
    out, mean, var = TropicalConvBNFn.apply(x, conv.weight, conv.weight2, conv.alpha, conv.beta, bn.weight, bn.bias,
                                            geom, bn.eps)
    with torch.no_grad():
        cnt = out.shape[0] * out.shape[2] * out.shape[3]
        m = bn.momentum if bn.momentum is not None else 0.1
        bn.running_mean.mul_(1 - m).add_(mean, alpha=m)
        bn.running_var.mul_(1 - m).add_(var * (cnt / max(cnt - 1, 1)), alpha=m)
        bn.num_batches_tracked += 1
    return out


class TropicalConv2d(nn.Module):
    """Tropical convolution layer with ``nn.Conv2d``'s constructor arguments.

    mode: "max_plus" | "min_plus" | "compound" | "parallel"; chan: "default" | "sum" | "max" | "min".
    params (compound / parallel; the paper's section "Specializations of compound/parallel tropical convolutions"): "2p" learnable alpha and beta
    per (c_out, c_in); "1p" complementary weights beta = 1 - alpha; "shared" beta = alpha;
    "opposite" beta = -alpha; "0p" alpha = beta = 1 (no scalars); "fixed" the constants
    ``fixed=(alpha, beta)``, e.g. (0.5, 0.5) or (1, -1), held as buffers.
    dtype: arithmetic type of the kernels ("f32" or "bf16"); parameters stay fp32."""

    PARAMS = ("0p", "1p", "2p", "shared", "opposite", "fixed")
    ND = 2          # spatial dimensions
    FN = None       # autograd Function of the layer (set below the class)

    def __init__(self, in_channels, out_channels, kernel_size, stride=1, padding=0, dilation=1,
                 bias=True, mode="compound", chan="default", params="2p", dtype="f32", fixed=(0.5, 0.5)):
        super().__init__()
        two = lambda v: (v,) * self.ND if isinstance(v, int) else tuple(v)
        self.kernel_size, self.stride, self.padding, self.dilation = map(two, (kernel_size, stride, padding, dilation))
        self.in_channels, self.out_channels = in_channels, out_channels
        self.mode, self.chan, self.params, self.dtype = mode, chan, params, dtype
        self.weight = nn.Parameter(torch.empty(out_channels, in_channels, *self.kernel_size))
        self.weight2 = nn.Parameter(torch.empty(out_channels, in_channels, *self.kernel_size)) if mode == "parallel" else None
        two_branch = mode in ("compound", "parallel")
        if params not in self.PARAMS:
            raise ValueError(f"params must be one of {self.PARAMS}")
        learn_a = two_branch and params in ("1p", "2p", "shared", "opposite")
        self.alpha = nn.Parameter(torch.empty(out_channels, in_channels)) if learn_a else None
        self.beta = nn.Parameter(torch.empty(out_channels, in_channels)) if two_branch and params == "2p" else None
        if two_branch and params == "fixed":
            self.register_buffer("alpha_fixed", torch.full((out_channels, in_channels), float(fixed[0])))
            self.register_buffer("beta_fixed", torch.full((out_channels, in_channels), float(fixed[1])))
        self.bias = nn.Parameter(torch.zeros(out_channels)) if bias else None
        self.reset_parameters()

    def reset_parameters(self):
        fan_in = self.in_channels * math.prod(self.kernel_size)
        bound = 1.0 / math.sqrt(fan_in)
        for w in (self.weight, self.weight2):
            if w is not None:
                nn.init.uniform_(w, -bound, bound)
        # the paper gives no initial values for alpha / beta: start from the normalised average of
        # the two branches divided by the fan-in of the channel sum
        for a in (self.alpha, self.beta):
            if a is not None:
                nn.init.constant_(a, 0.5 / self.in_channels)

    def extra_repr(self):
        return (f"{self.in_channels}, {self.out_channels}, kernel_size={self.kernel_size}, stride={self.stride}, "
                f"padding={self.padding}, dilation={self.dilation}, mode={self.mode}, chan={self.chan}, "
                f"params={self.params}, dtype={self.dtype}")

    def forward(self, x):
        alpha, beta = self.alpha, self.beta
        if self.mode in ("compound", "parallel"):
            if self.params == "1p":
                beta = 1.0 - alpha
            elif self.params == "shared":
                beta = alpha
            elif self.params == "opposite":
                beta = -alpha
            elif self.params == "fixed":
                alpha, beta = self.alpha_fixed, self.beta_fixed
        geom = (self.mode, self.chan, self.dtype, self.stride, self.padding, self.dilation)
        return self.FN.apply(x, self.weight, self.weight2, alpha, beta, self.bias, geom)


TropicalConv2d.FN = TropicalConvFn


class TropicalBasicBlock(nn.Module):
    """The paper's TCNN basic block 2: Tropical - BN - Tropical - BN, intermediate ReLU removed,
    identity (or 1x1 standard-convolution) shortcut, ReLU after the sum."""

    def __init__(self, cin, cout, stride, mode, dtype, fused_bn=False):
        super().__init__()
        self.fused_bn = fused_bn    # batch-normalisation statistics from the tropical kernels' epilogue
        self.conv1 = TropicalConv2d(cin, cout, 3, stride=stride, padding=1, bias=False, mode=mode, dtype=dtype)
        self.bn1 = nn.BatchNorm2d(cout)
        self.conv2 = TropicalConv2d(cout, cout, 3, stride=1, padding=1, bias=False, mode=mode, dtype=dtype)
        self.bn2 = nn.BatchNorm2d(cout)
        self.down = None
        if stride != 1 or cin != cout:
            self.down = nn.Sequential(nn.Conv2d(cin, cout, 1, stride=stride, bias=False), nn.BatchNorm2d(cout))

    def forward(self, x):
        if self.fused_bn:
            out = tropical_conv_bn(self.conv2, self.bn2, tropical_conv_bn(self.conv1, self.bn1, x))
        else:
            out = self.bn2(self.conv2(self.bn1(self.conv1(x))))
        return torch.relu(out + (x if self.down is None else self.down(x)))


class StandardBasicBlock(nn.Module):
    def __init__(self, cin, cout, stride):
        super().__init__()
        self.conv1 = nn.Conv2d(cin, cout, 3, stride=stride, padding=1, bias=False)
        self.bn1 = nn.BatchNorm2d(cout)
        self.conv2 = nn.Conv2d(cout, cout, 3, padding=1, bias=False)
        self.bn2 = nn.BatchNorm2d(cout)

    def forward(self, x):
        return torch.relu(self.bn2(self.conv2(torch.relu(self.bn1(self.conv1(x))))) + x)


class HybridResNet18(nn.Module):
    """ResNet-18 shape; every 3x3 convolution of stages 2-4 is a tropical layer of the given mode
    (stem, stage 1 and the 1x1 downsamples are standard convolutions)."""

    def __init__(self, mode="compound", dtype="bf16", num_classes=1000, fused_bn=False):
        super().__init__()
        self.stem = nn.Sequential(nn.Conv2d(3, 64, 7, stride=2, padding=3, bias=False), nn.BatchNorm2d(64),
                                  nn.ReLU(inplace=True), nn.MaxPool2d(3, stride=2, padding=1))
        self.layer1 = nn.Sequential(StandardBasicBlock(64, 64, 1), StandardBasicBlock(64, 64, 1))
        self.layer2 = nn.Sequential(TropicalBasicBlock(64, 128, 2, mode, dtype, fused_bn), TropicalBasicBlock(128, 128, 1, mode, dtype, fused_bn))
        self.layer3 = nn.Sequential(TropicalBasicBlock(128, 256, 2, mode, dtype, fused_bn), TropicalBasicBlock(256, 256, 1, mode, dtype, fused_bn))
        self.layer4 = nn.Sequential(TropicalBasicBlock(256, 512, 2, mode, dtype, fused_bn), TropicalBasicBlock(512, 512, 1, mode, dtype, fused_bn))
        self.head = nn.Sequential(nn.AdaptiveAvgPool2d(1), nn.Flatten(), nn.Linear(512, num_classes))

    def forward(self, x):
        x = self.layer1(self.stem(x))
        x = self.layer4(self.layer3(self.layer2(x)))
        return self.head(x)

    def tropical_layers(self):
        return [m for m in self.modules() if isinstance(m, TropicalConv2d)]


class TropicalDepthwiseFn(torch.autograd.Function):
    """Depthwise (groups = C) form over tconv_dw_forward / tconv_dw_backward; see TropicalConvFn."""

    @staticmethod
    def forward(ctx, x, w, w2, alpha, beta, bias, geom):
        mode, dtype, stride, pad, dil = geom
        dt = tconv.TORCH_DTYPE[dtype]
        N, C, H, W = x.shape
        _, R, S = w.shape
        d = dict(N=N, C=C, H=H, W=W, K=C, R=R, S=S, stride_h=stride[0], stride_w=stride[1],
                 pad_h=pad[0], pad_w=pad[1], dil_h=dil[0], dil_w=dil[1], mode=mode, chan="sum", dtype=dtype)
        xc = x.detach().to(dt).contiguous()
        wc = w.detach().to(dt).contiguous()
        w2c = w2.detach().to(dt).contiguous() if w2 is not None else None
        al = alpha.detach().float().contiguous() if alpha is not None else None
        be = beta.detach().float().contiguous() if beta is not None else None
        bi = bias.detach().float().contiguous() if bias is not None else None
        need_grad = any(t is not None and t.requires_grad for t in (x, w, w2, alpha, beta, bias))
        y, winners = tconv.dw_forward(d, xc, wc, w2c, al, be, bi, want_winners=need_grad)
        ctx.d, ctx.in_dtype = d, x.dtype
        ctx.save_for_backward(xc, wc, w2c, al, be, winners)
        ctx.has = (w2 is not None, alpha is not None, beta is not None, bias is not None)
        return y.to(x.dtype) if x.dtype != dt else y

    @staticmethod
    def backward(ctx, gy):
        xc, wc, w2c, al, be, winners = ctx.saved_tensors
        d = ctx.d
        g = gy.to(tconv.TORCH_DTYPE[d["dtype"]]).contiguous()
        grads = tconv.dw_backward(d, xc, wc, g, w2c, al, be, winners)
        has_w2, has_a, has_b, has_bias = ctx.has
        return (grads["grad_x"].to(ctx.in_dtype), grads["grad_w"], grads.get("grad_w2") if has_w2 else None,
                grads.get("grad_alpha") if has_a else None, grads.get("grad_beta") if has_b else None,
                grads["grad_bias"] if has_bias else None, None)


class TropicalDepthwiseConv2d(nn.Module):
    """Depthwise tropical convolution (``nn.Conv2d(channels, channels, k, groups=channels)``'s place in
    a MobileNetV2 block): per channel one window of weights, one alpha and one beta.

    mode and params as in TropicalConv2d ("2p", "1p", "shared", "opposite", "0p", "fixed")."""

    def __init__(self, channels, kernel_size, stride=1, padding=0, dilation=1, bias=True,
                 mode="compound", params="2p", dtype="f32", fixed=(0.5, 0.5)):
        super().__init__()
        two = lambda v: (v, v) if isinstance(v, int) else tuple(v)
        self.kernel_size, self.stride, self.padding, self.dilation = map(two, (kernel_size, stride, padding, dilation))
        self.channels, self.mode, self.params, self.dtype = channels, mode, params, dtype
        if params not in TropicalConv2d.PARAMS:
            raise ValueError(f"params must be one of {TropicalConv2d.PARAMS}")
        R, S = self.kernel_size
        self.weight = nn.Parameter(torch.empty(channels, R, S))
        self.weight2 = nn.Parameter(torch.empty(channels, R, S)) if mode == "parallel" else None
        two_branch = mode in ("compound", "parallel")
        self.alpha = nn.Parameter(torch.empty(channels)) if two_branch and params in ("1p", "2p", "shared", "opposite") else None
        self.beta = nn.Parameter(torch.empty(channels)) if two_branch and params == "2p" else None
        if two_branch and params == "fixed":
            self.register_buffer("alpha_fixed", torch.full((channels,), float(fixed[0])))
            self.register_buffer("beta_fixed", torch.full((channels,), float(fixed[1])))
        self.bias = nn.Parameter(torch.zeros(channels)) if bias else None
        bound = 1.0 / math.sqrt(R * S)
        for w in (self.weight, self.weight2):
            if w is not None:
                nn.init.uniform_(w, -bound, bound)
        for a in (self.alpha, self.beta):
            if a is not None:
                nn.init.constant_(a, 0.5)

    def extra_repr(self):
        return (f"{self.channels}, kernel_size={self.kernel_size}, stride={self.stride}, padding={self.padding}, "
                f"dilation={self.dilation}, mode={self.mode}, params={self.params}, dtype={self.dtype}")

    def forward(self, x):
        alpha, beta = self.alpha, self.beta
        if self.mode in ("compound", "parallel"):
            if self.params == "1p":
                beta = 1.0 - alpha
            elif self.params == "shared":
                beta = alpha
            elif self.params == "opposite":
                beta = -alpha
            elif self.params == "fixed":
                alpha, beta = self.alpha_fixed, self.beta_fixed
        geom = (self.mode, self.dtype, self.stride, self.padding, self.dilation)
        return TropicalDepthwiseFn.apply(x, self.weight, self.weight2, alpha, beta, self.bias, geom)


class TropicalConv3dFn(torch.autograd.Function):
    """y = tconv3d_forward(...); backward = tconv3d_backward with the stored winners."""

    @staticmethod
    def forward(ctx, x, w, w2, alpha, beta, bias, geom):
        from . import tconv3d
        mode, chan, dtype, stride, pad, dil = geom
        dt = tconv.TORCH_DTYPE[dtype]
        N, C, D, H, W = x.shape
        K, _, T, R, S = w.shape
        d = dict(N=N, C=C, D=D, H=H, W=W, K=K, T=T, R=R, S=S, stride=tuple(stride), pad=tuple(pad),
                 dil=tuple(dil), mode=mode, chan=chan, dtype=dtype)
        cast = lambda t, ty: t.detach().to(ty).contiguous() if t is not None else None
        xc, wc, w2c = cast(x, dt), cast(w, dt), cast(w2, dt)
        al, be, bi = cast(alpha, torch.float32), cast(beta, torch.float32), cast(bias, torch.float32)
        need_grad = any(t is not None and t.requires_grad for t in (x, w, w2, alpha, beta, bias))
        y, winners = tconv3d.forward(d, xc, wc, w2c, al, be, bi, want_winners=need_grad)
        ctx.d, ctx.in_dtype = d, x.dtype
        ctx.save_for_backward(xc, wc, w2c, al, be, winners)
        ctx.has = (w2 is not None, alpha is not None, beta is not None, bias is not None)
        return y.to(x.dtype) if x.dtype != dt else y

    @staticmethod
    def backward(ctx, gy):
        from . import tconv3d
        xc, wc, w2c, al, be, winners = ctx.saved_tensors
        d = ctx.d
        g = gy.detach().to(tconv.TORCH_DTYPE[d["dtype"]]).contiguous()
        grads = tconv3d.backward(d, xc, wc, g, w2c, al, be, winners, need_grad_x=ctx.needs_input_grad[0])
        has_w2, has_a, has_b, has_bias = ctx.has
        gx = grads["grad_x"].to(ctx.in_dtype) if "grad_x" in grads else None
        return (gx, grads["grad_w"], grads.get("grad_w2") if has_w2 else None,
                grads.get("grad_alpha") if has_a else None, grads.get("grad_beta") if has_b else None,
                grads["grad_bias"] if has_bias else None, None)


class TropicalConv3d(TropicalConv2d):
    """Three-dimensional tropical convolution (Section 3.2 and the Conv3d forms of Sections 3.4 / 3.5)
    with ``nn.Conv3d``'s constructor arguments; input [N, C, D, H, W]; mode / chan / params / dtype
    as in TropicalConv2d.  Windows of up to 256 taps (the paper's 3-D LeNet uses 5 x 5 x 5)."""

    ND = 3
    FN = TropicalConv3dFn


class TropicalConv1d(nn.Module):
    """1-D tropical convolution (Section 3.2) with ``nn.Conv1d``'s constructor arguments; mode / chan /
    params / dtype as in TropicalConv2d.  The length-3, stride-1 layers run as 1 x 3 windows on a signal
    of unit height through the tiled 2-D kernels; every other window (up to 256 taps; the paper's audio
    networks open with length 80 at stride 4) goes as a 1 x 1 x k window through the three-dimensional
    entry points, which run windows of four taps or more at stride 1, 2 or 4 (no dilation) on their
    one-dimensional kernels and the rest on the any-shape kernels."""

    def __init__(self, in_channels, out_channels, kernel_size, stride=1, padding=0, dilation=1,
                 bias=True, mode="compound", chan="default", params="2p", dtype="f32", fixed=(0.5, 0.5)):
        super().__init__()
        self.tiled = (kernel_size == 3 and stride == 1 and dilation == 1)
        if self.tiled:
            self.conv = TropicalConv2d(in_channels, out_channels, (1, kernel_size), stride=(1, stride),
                                       padding=(0, padding), dilation=(1, dilation), bias=bias, mode=mode,
                                       chan=chan, params=params, dtype=dtype, fixed=fixed)
        else:
            self.conv = TropicalConv3d(in_channels, out_channels, (1, 1, kernel_size), stride=(1, 1, stride),
                                       padding=(0, 0, padding), dilation=(1, 1, dilation), bias=bias, mode=mode,
                                       chan=chan, params=params, dtype=dtype, fixed=fixed)

    def forward(self, x):                      # x: [N, C, L]
        if self.tiled:
            return self.conv(x.unsqueeze(2)).squeeze(2)
        return self.conv(x[:, :, None, None, :])[:, :, 0, 0, :]
