"""Data-parallel combination of per-rank training steps (the paper's "XLA GSPMD partitioning" section: data
parallelism with replicated parameters), one process per GPU over torch.distributed.

Every rank runs t5_train_step_fwd_bwd on its own batch rows.  The step normalises by the rank's own count of
non-pad targets W_r, the job's loss normalises by W = sum_r W_r, so
    L = sum_r (W_r / W) L_r          and          dL/dtheta = sum_r (W_r / W) dL_r/dtheta.
combine() does exactly that: one all-reduce of W (a scalar), a scaling of the local gradient buffer by W_r / W, and
a sum all-reduce of the flat gradient buffer in buckets issued asynchronously from the end of the buffer (the
decoder's and the last layers' gradients, which the backward pass finishes first) to its start.  This module holds no
model arithmetic beyond that weighting; the buffers may live on any device the process group's backend serves
(NCCL for CUDA tensors, gloo for CPU tensors in the tests).
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def bucket_ranges(n_elements: int, bucket_elements: int):
    """[(begin, end)] covering [0, n) from the END of the buffer to its start, each at most bucket_elements long."""
    if bucket_elements < 1:
        raise ValueError("bucket_elements must be positive")
    out, hi = [], n_elements
    while hi > 0:
        lo = max(0, hi - bucket_elements)
        out.append((lo, hi))
        hi = lo
    return out


def combine(grads: torch.Tensor, loss4: torch.Tensor, group=None, bucket_elements: int = 64 * 1024 * 1024):
    """In place: grads <- sum_r (W_r / W) grads_r; loss4 <- [L, ce, z-part, W] of the whole job.

    grads: the rank's flat float32 gradient buffer; loss4: its [L_r, ce_r, z_r, W_r] as the step wrote it.
    Returns the job's W (a Python float).  With W = 0 (no target anywhere) everything becomes zero."""
    if not dist.is_initialized() or dist.get_world_size(group) == 1:
        return float(loss4[3].item())
    w_local = loss4[3:4].clone()
    w_total = w_local.clone()
    dist.all_reduce(w_total, op=dist.ReduceOp.SUM, group=group)
    scale = torch.where(w_total > 0, w_local / torch.clamp(w_total, min=1.0), torch.zeros_like(w_local))
    grads.mul_(scale.to(grads.dtype))
    pending = []
    for lo, hi in bucket_ranges(grads.numel(), bucket_elements):
        pending.append(dist.all_reduce(grads[lo:hi], op=dist.ReduceOp.SUM, group=group, async_op=True))
    parts = loss4[:3] * scale
    dist.all_reduce(parts, op=dist.ReduceOp.SUM, group=group)
    for p in pending:
        p.wait()
    loss4[:3] = parts
    loss4[3:4] = w_total
    return float(w_total.item())
