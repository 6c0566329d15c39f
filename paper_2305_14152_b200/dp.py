"""Data-parallel plumbing for the scale gradients (torch.distributed only; no arithmetic of the
method lives here).

The layer shards along tokens: every rank holds the full frozen Q, z and the scales (they are
small -- that is the point of Sec. 3.2 / 3.3), Y and dX rows are independent per token, and the
scale gradient of Eq. 2 is a sum over tokens.  So the one exchange of a data-parallel step is an
all-reduce (sum) of dS over the ranks, after which every rank applies the same AdamW step
(App. A) to its copy of the scales.  All dS tensors of a layer travel in one flat bucket: on
NVSwitch the cost of a collective is launch latency, not link count, so one call per layer
beats one per linear.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def bucket_views(tensors, bucket=None):
    """A flat fp32 bucket with room for every tensor of `tensors` and, per tensor, the view of the
    bucket that has its shape.  Offsets are rounded up to 64 elements (256 bytes) so that every
    view can be handed to the library as an aligned dS pointer."""
    offs, total = [], 0
    for t in tensors:
        offs.append(total)
        total += (t.numel() + 63) // 64 * 64
    if bucket is None:
        bucket = torch.zeros(total, dtype=torch.float32, device=tensors[0].device)
    elif bucket.numel() < total or bucket.dtype != torch.float32:
        raise ValueError("bucket too small or not fp32")
    views = [bucket[o:o + t.numel()].view(t.shape) for o, t in zip(offs, tensors)]
    return bucket, views


def allreduce_scale_grads(grads, group=None, average=False, bucket=None):
    """Sums (or averages) every tensor of `grads` over the ranks of `group`, in place, with one
    all-reduce of a flat bucket.  A step whose kernels already wrote dS into bucket_views() of
    `bucket` passes that bucket and skips both copies."""
    if not dist.is_available() or not dist.is_initialized():
        return grads
    if bucket is not None and all(g.untyped_storage().data_ptr() == bucket.untyped_storage().data_ptr()
                                  for g in grads):
        flat, views = bucket, None
    else:
        flat, views = bucket_views(grads, bucket)
        for v, g in zip(views, grads):
            v.copy_(g)
    dist.all_reduce(flat, op=dist.ReduceOp.SUM, group=group)
    if average:
        flat.div_(dist.get_world_size(group))
    if views is not None:
        for v, g in zip(views, grads):
            g.copy_(v)
    return grads


def layer_train_step_dp(linears, lr, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0, step=1,
                        group=None, average=False, bucket=None):
    """One data-parallel step of a layer: forward, dX and dS of every linear on this rank's tokens
    (one library call, no optimizer step), one all-reduce of all dS, then the AdamW step on every
    rank's scales.  When the linears' dS tensors are bucket_views() of `bucket`, nothing is copied."""
    from . import binding
    binding.layer_train_step(linears, apply_adamw=False)
    allreduce_scale_grads([L.dS for L in linears], group=group, average=average, bucket=bucket)
    for L in linears:
        binding.scale_adamw(L.w.scales, L.dS, L.m, L.v, lr, beta1, beta2, eps, weight_decay, step)
