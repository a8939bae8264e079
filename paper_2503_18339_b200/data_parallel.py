"""Batch-sharded channel-wise fake-quantization: every rank holds a slice of the batch and all ranks
quantize with ONE per-channel range, that of the whole batch (Eq. 4 over the global batch).

The path has exactly one exchange step, between the range (Eq. 4) and the scale / zero-point
(Eq. 5): the per-group minima and maxima (G floats each) are all-reduced, MIN and MAX.  Everything
before and after is local.  The exchange uses `torch.distributed` (NCCL on GPUs, gloo on CPU) on the
buffers the library wrote, in place; no arithmetic happens outside the library and the collective.

Without this module each rank quantizes with the range of its own slice (independent replicas),
which is what `bench.py --gpus N` times.
"""
from __future__ import annotations

from typing import Optional

import torch
import torch.distributed as dist


def sync_range(lo: torch.Tensor, hi: torch.Tensor, group=None, stream=None) -> None:
    """In place: lo <- min over ranks, hi <- max over ranks (two all-reduces of G floats, issued back to
    back; the messages are a few KB, so both are latency-bound).  On CUDA tensors the collectives are
    ordered after what `stream` holds - the range kernel that wrote lo / hi - and the stream then waits
    for them.  A no-op without an initialised process group or with a single rank."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return
    if lo.is_cuda and stream is not None:
        with torch.cuda.stream(stream):       # the process group orders its work after the current stream
            dist.all_reduce(lo, op=dist.ReduceOp.MIN, group=group)
            dist.all_reduce(hi, op=dist.ReduceOp.MAX, group=group)
        return
    dist.all_reduce(lo, op=dist.ReduceOp.MIN, group=group)
    dist.all_reduce(hi, op=dist.ReduceOp.MAX, group=group)


def fakequant_forward(x: torch.Tensor, bits: int, channel_axis: int = 1, group_mode: int = 0, group=None,
                      stream=None):
    """Forward of a training step on this rank's slice: local range -> all-reduce -> y and the packed
    STE mask with the global range.  Returns the binding's FakeQuantOut (y, packed_mask, lo, hi)."""
    from . import binding as b
    lo, hi = b.granq_range(x, channel_axis=channel_axis, group=group_mode, stream=stream)
    sync_range(lo, hi, group, stream)
    return b.granq_fakequant_fwd_packmask(x, bits, lo, hi, channel_axis=channel_axis, group=group_mode,
                                          stream=stream)


def fakequant_backward(gy: torch.Tensor, packed_mask: torch.Tensor, gx: Optional[torch.Tensor] = None, stream=None):
    """Backward of the same step: purely local, from the mask the forward pass stored."""
    from . import binding as b
    return b.granq_fakequant_bwd_packmask(gy, packed_mask, gx=gx, stream=stream)
