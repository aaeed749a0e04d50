"""Host-side helpers for running the step on several ranks (one process per GPU).

Two deployment shapes (Algorithm 1 assumes M data-parallel replicas that share the optimizer's
random state):

* replicas -- every rank holds the full buffers and runs the identical step; nothing here is needed,
  the results agree bit for bit because the noise depends only on (seed, step, tensor_id, index).
* shards -- every rank owns one contiguous slice.  ``partition`` gives the slices (multiples of 8
  elements, so every slice starts on a noise-group boundary and a 16-byte boundary); each rank calls
  ``sr_adamw_step`` with ``elem_offset`` = start of its slice.  The only exchange is the squared
  gradient norm: ``global_sqnorm`` all-gathers one double per rank and adds them in rank order, so
  every rank obtains the same bits whatever the collective's internal order.

Works with any torch.distributed backend (NCCL on GPUs, gloo on CPU for tests).
"""

from __future__ import annotations

from typing import List, Tuple

import torch
import torch.distributed as dist


def partition(n: int, world_size: int, align: int = 8) -> List[Tuple[int, int]]:
    """Contiguous (start, length) per rank; all starts are multiples of ``align``; the last rank
    takes the ragged remainder.  Ranks beyond the data get empty slices."""
    if n < 0 or world_size < 1 or align < 1:
        raise ValueError("bad arguments")
    per = -(-n // world_size)                 # ceil
    per = -(-per // align) * align            # round up to the alignment
    out = []
    for r in range(world_size):
        start = min(r * per, n)
        out.append((start, min(per, n - start)))
    return out


def global_sqnorm(local_sqnorm: torch.Tensor, group=None) -> torch.Tensor:
    """local_sqnorm: one float64 (this rank's ``grad_sqnorm`` result, on the device the backend
    uses).  Returns the sum over ranks, added in rank order 0, 1, ... in float64: identical bits on
    every rank."""
    if local_sqnorm.dtype != torch.float64 or local_sqnorm.numel() != 1:
        raise TypeError("expected one float64")
    world = dist.get_world_size(group)
    parts = [torch.empty_like(local_sqnorm) for _ in range(world)]
    dist.all_gather(parts, local_sqnorm.contiguous(), group=group)
    total = parts[0].clone()
    for t in parts[1:]:
        total = total + t
    return total


def max_over_ranks(value: float, device, group=None) -> float:
    """Largest value over ranks (used for timings)."""
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return float(t.item())
