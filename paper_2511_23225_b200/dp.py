"""The one exchange the method needs under data parallelism (plumbing over torch.distributed, no arithmetic of the
method): per-tensor scaling means ONE scale for the whole tensor (Sec. 4.3), so when the tokens of a tensor are
sharded over ranks, the per-rank amax values a step produced are MAX-reduced before they enter the amax histories --
a few floats per step, off the critical path under delayed scaling (this step's amax only sets the next step's
scale).  The library calls themselves exchange nothing: every rank casts and multiplies its own shard.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def allreduce_amax(amax: torch.Tensor, group=None) -> torch.Tensor:
    """MAX all-reduce, in place, of a float32 tensor of per-tensor amax values (one entry per quantised tensor; the
    same order on every rank).  Identity without an initialised process group or with a single rank.  NCCL for CUDA
    tensors, gloo for CPU tensors: whatever backend the group was made with."""
    if amax.dtype != torch.float32:
        raise TypeError("amax values are float32")
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(amax, op=dist.ReduceOp.MAX, group=group)
    return amax
