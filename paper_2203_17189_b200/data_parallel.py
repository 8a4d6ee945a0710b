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


class _DeviceFloat:
    """A float32 scalar at a raw device address, for torch.as_tensor (CUDA array interface)."""

    def __init__(self, ptr):
        self.__cuda_array_interface__ = {"shape": (1,), "typestr": "<f4", "data": (int(ptr), False), "version": 2}


class OverlappedReducer:
    """Gradient all-reduce that runs while the backward pass is still going.

    The library reports each range of the gradient buffer as soon as its last write is enqueued (t5_set_grad_hook).
    For every range this class multiplies the rank's values by W_r (the rank's target count, read on the device), and
    starts a sum all-reduce on a communication stream behind an event recorded on the stream the library names;
    nothing blocks the host or the compute streams.  finish() then waits for the collectives, all-reduces W and the
    loss parts, and divides by the job's W:  grads <- sum_r W_r g_r / W,  loss4 <- [L, ce, z-part, W] of the job -
    the same result as combine().  reduce_range() is the hook body and can be driven by hand (CPU tensors, gloo)."""

    def __init__(self, grads: torch.Tensor, group=None):
        self.grads, self.group = grads, group
        self.comm = torch.cuda.Stream(device=grads.device) if grads.is_cuda else None
        self.pending, self.ranges = [], []

    def attach(self, handle):
        handle.t5_set_grad_hook(self._hook)
        return self

    def _hook(self, offset, count, weight_ptr, stream_ptr):
        w = torch.as_tensor(_DeviceFloat(weight_ptr), device=self.grads.device)
        self.reduce_range(offset, count, w, stream_ptr)

    def reduce_range(self, offset, count, rank_weight, stream_ptr=None):
        """rank_weight: one-element float32 tensor on the gradients' device holding W_r."""
        self.ranges.append((int(offset), int(count)))
        view = self.grads[offset:offset + count]
        active = dist.is_initialized() and dist.get_world_size(self.group) > 1
        if self.comm is None:
            view.mul_(rank_weight)
            if active:
                self.pending.append(dist.all_reduce(view, op=dist.ReduceOp.SUM, group=self.group, async_op=True))
            return
        ready = torch.cuda.Event()
        if stream_ptr:
            ready.record(torch.cuda.ExternalStream(int(stream_ptr), device=self.grads.device))
        else:       # a null handle is the default stream
            ready.record(torch.cuda.default_stream(self.grads.device))
        self.comm.wait_event(ready)
        with torch.cuda.stream(self.comm):
            view.mul_(rank_weight)
            if active:
                self.pending.append(dist.all_reduce(view, op=dist.ReduceOp.SUM, group=self.group, async_op=True))

    def finish(self, loss4: torch.Tensor):
        """Call after t5_train_step_fwd_bwd returned (on the stream it was given).  Returns the job's W."""
        for work in self.pending:
            work.wait()
        self.pending = []
        if self.comm is not None:
            torch.cuda.current_stream(self.grads.device).wait_stream(self.comm)
        active = dist.is_initialized() and dist.get_world_size(self.group) > 1
        w_total = loss4[3:4].clone()
        parts = loss4[:3] * loss4[3:4]
        if active:
            dist.all_reduce(w_total, op=dist.ReduceOp.SUM, group=self.group)
            dist.all_reduce(parts, op=dist.ReduceOp.SUM, group=self.group)
        inv = torch.where(w_total > 0, 1.0 / torch.clamp(w_total, min=1.0), torch.zeros_like(w_total))
        self.grads.mul_(inv.to(self.grads.dtype))
        loss4[:3] = parts * inv
        loss4[3:4] = w_total
        covered = sorted(self.ranges)
        self.ranges = []
        return float(w_total.item()), covered
