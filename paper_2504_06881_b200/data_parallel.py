"""Data-parallel training over batch shards (one process per GPU).

The tropical layers shard over the batch with no exchange in the forward or in grad_x: every
output depends on one image only.  The parameter gradients (grad_w, grad_w2, grad_alpha,
grad_beta, grad_bias and those of the surrounding standard layers) are sums over the batch, so a
step needs exactly one exchange: a sum of the parameter gradients over the ranks.  This module does
that exchange with ``torch.distributed`` (NCCL on GPUs, gloo on CPU): the gradients are packed into
one flat fp32 buffer per call, so that a network costs one all-reduce, and averaged or summed.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def all_reduce_gradients(parameters, group=None, average=True):
    """Sum (or average) the ``.grad`` of every parameter over the ranks of `group`, in place.

    Parameters without a gradient on this rank contribute zeros (every rank must walk the same
    parameter list).  Returns the number of elements exchanged."""
    params = [p for p in parameters]
    if not params:
        return 0
    if not dist.is_available() or not dist.is_initialized():
        raise RuntimeError("all_reduce_gradients needs an initialised torch.distributed process group")
    dev = params[0].device
    flat = torch.zeros(sum(p.numel() for p in params), dtype=torch.float32, device=dev)
    off = 0
    for p in params:
        if p.grad is not None:
            flat[off:off + p.numel()].copy_(p.grad.reshape(-1))
        off += p.numel()
    dist.all_reduce(flat, op=dist.ReduceOp.SUM, group=group)
    if average:
        flat /= dist.get_world_size(group)
    off = 0
    for p in params:
        g = flat[off:off + p.numel()].view_as(p).to(p.dtype)
        if p.grad is None:
            p.grad = g.clone()
        else:
            p.grad.copy_(g)
        off += p.numel()
    return flat.numel()


def shard_batch(x, rank=None, world=None):
    """This rank's contiguous slice of a batch (dimension 0), sizes differing by at most one."""
    rank = dist.get_rank() if rank is None else rank
    world = dist.get_world_size() if world is None else world
    n = x.shape[0]
    lo = (n * rank) // world
    hi = (n * (rank + 1)) // world
    return x[lo:hi]
