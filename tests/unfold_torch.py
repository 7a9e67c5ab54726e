"""The paper's PyTorch-only formulation of the compound / parallel layers (appendix
"Implementation Without TileLang": unfold -> add / min / max -> channel operations), written
with torch tensor primitives and chunked over output channels to bound memory.  Used only as a
second formulation for whole-network consistency checks; it shares nothing with the library."""
import torch
import torch.nn.functional as F


def tropical_unfold(x, w, w2, alpha, beta, stride, padding, dilation, chunk=8):
    """x [N,C,H,W], w/w2 [K,C,R,S] (same dtype: each tap sum is one rounded add in that dtype);
    alpha/beta [K,C] fp32.  Returns fp32 y [N,K,OH,OW] = sum_c alpha*min + beta*max."""
    N, C, H, W = x.shape
    K, _, R, S = w.shape
    OH = (H + 2 * padding - dilation * (R - 1) - 1) // stride + 1
    OW = (W + 2 * padding - dilation * (S - 1) - 1) // stride + 1
    p = F.unfold(x, (R, S), dilation=dilation, padding=padding, stride=stride)      # [N, C*R*S, P]
    p = p.view(N, 1, C, R * S, OH * OW)
    out = torch.empty(N, K, OH * OW, dtype=torch.float32, device=x.device)
    for k0 in range(0, K, chunk):
        k1 = min(K, k0 + chunk)
        t1 = p + w[k0:k1].reshape(1, k1 - k0, C, R * S, 1)
        mn = t1.amin(dim=3).float()
        t2 = t1 if w2 is None else p + w2[k0:k1].reshape(1, k1 - k0, C, R * S, 1)
        mx = t2.amax(dim=3).float()
        a = alpha[k0:k1].view(1, k1 - k0, C, 1)
        b = beta[k0:k1].view(1, k1 - k0, C, 1)
        out[:, k0:k1] = (a * mn + b * mx).sum(dim=2)
    return out.view(N, K, OH, OW)
