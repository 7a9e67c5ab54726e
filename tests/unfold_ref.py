"""Second, independent formulation of the tropical layers used to pin the oracle.

It follows the three steps the paper gives for its PyTorch-only back end
(appendix "Implementation Without TileLang"): unfold the input into patches,
broadcast-add the weight and take min / max over the window axis with library
routines, then combine over input channels.  numpy's argmin / argmax return the
first occurrence, which is the lowest-tap tie rule.  Written with numpy only; it
calls nothing from the oracle or from the CUDA package.
"""
import numpy as np


def out_hw(d):
    def ext(i, p, dl, k, s):
        span = i + 2 * p - dl * (k - 1) - 1
        return 0 if span < 0 else span // s + 1
    return (ext(d["H"], d["pad_h"], d["dil_h"], d["R"], d["stride_h"]),
            ext(d["W"], d["pad_w"], d["dil_w"], d["S"], d["stride_w"]))


def unfold(d, x, fill=0.0):
    """patches[N, C, R*S, OH, OW]; the padding holds `fill` (zero padding by default)."""
    OH, OW = out_hw(d)
    N, C, H, W, R, S = d["N"], d["C"], d["H"], d["W"], d["R"], d["S"]
    xp = np.full((N, C, H + 2 * d["pad_h"], W + 2 * d["pad_w"]), fill, x.dtype)
    xp[:, :, d["pad_h"]:d["pad_h"] + H, d["pad_w"]:d["pad_w"] + W] = x
    p = np.empty((N, C, R * S, OH, OW), x.dtype)
    for r in range(R):
        for s in range(S):
            h0, w0 = r * d["dil_h"], s * d["dil_w"]
            p[:, :, r * S + s] = xp[:, :, h0:h0 + (OH - 1) * d["stride_h"] + 1:d["stride_h"],
                                    w0:w0 + (OW - 1) * d["stride_w"] + 1:d["stride_w"]]
    return p


def fmaf32(a, b, c):
    """float32 fused multiply-add emulated in float64 (the product of two float32
    is exact in float64; the final double rounding is harmless for the test data)."""
    return (a.astype(np.float64) * b.astype(np.float64) + c.astype(np.float64)).astype(np.float32)


def forward(d, x, w, w2=None, alpha=None, beta=None, bias=None):
    """fp32 forward.  Returns y, idx (Max/Min combine) or codes (Sum combine)."""
    N, C, K, R, S = d["N"], d["C"], d["K"], d["R"], d["S"]
    OH, OW = out_hw(d)
    mode, chan = d["mode"], d["chan"]
    if chan == "default":
        chan = {"max_plus": "max", "min_plus": "min"}.get(mode, "sum")
    neutral = d.get("pad_mode", "zero") == "neutral"
    wr = w.astype(np.float32).reshape(K, C, R * S)
    wr2 = w2.astype(np.float32).reshape(K, C, R * S) if mode == "parallel" else wr
    if not neutral:
        p = unfold(d, x.astype(np.float32))                  # [N,C,RS,OH,OW]
        t1 = p[:, None] + wr[None, :, :, :, None, None]      # [N,K,C,RS,OH,OW], float32 adds
        t2 = p[:, None] + wr2[None, :, :, :, None, None] if mode == "parallel" else t1
    else:
        # neutral padding: the padding holds the identity of each branch's semiring, so a padded
        # tap sum is +inf in the min branch and -inf in the max branch and never wins
        t1 = unfold(d, x.astype(np.float32), np.inf)[:, None] + wr[None, :, :, :, None, None]
        t2 = unfold(d, x.astype(np.float32), -np.inf)[:, None] + wr2[None, :, :, :, None, None]
    mn, amn = t1.min(axis=3), t1.argmin(axis=3)              # [N,K,C,OH,OW]
    mx, amx = t2.max(axis=3), t2.argmax(axis=3)
    idx = codes = None
    if mode in ("compound", "parallel"):
        a = np.ones((K, C), np.float32) if alpha is None else alpha.astype(np.float32)
        b = np.ones((K, C), np.float32) if beta is None else beta.astype(np.float32)
        acc = np.zeros((N, K, OH, OW), np.float32)
        for c in range(C):
            acc = fmaf32(np.broadcast_to(a[None, :, c, None, None], acc.shape), mn[:, :, c], acc)
            acc = fmaf32(np.broadcast_to(b[None, :, c, None, None], acc.shape), mx[:, :, c], acc)
        y = acc
        codes = (amn | (amx << 4)).astype(np.uint8)
    else:
        m, am = (mn, amn) if mode == "min_plus" else (mx, amx)
        if chan == "sum":
            acc = np.zeros((N, K, OH, OW), np.float32)
            for c in range(C):
                acc = acc + m[:, :, c]
            y = acc
            codes = (am if mode == "min_plus" else (am << 4)).astype(np.uint8)
        else:
            cs = m.argmax(axis=2) if chan == "max" else m.argmin(axis=2)   # first c on ties
            y = np.take_along_axis(m, cs[:, :, None], axis=2)[:, :, 0]
            tap = np.take_along_axis(am, cs[:, :, None], axis=2)[:, :, 0]
            idx = (cs * (R * S) + tap).astype(np.int32)
    if bias is not None:
        y = y + bias.astype(np.float32)[None, :, None, None]
    return y.astype(np.float32), idx, codes
