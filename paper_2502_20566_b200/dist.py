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


def wire_bytes(n: int, world_size: int, grad_dtype: torch.dtype) -> dict:
    """Bytes one rank sends per iteration of ``sharded_clipped_step`` on a buffer of n elements: the
    reduce-scatter of the gradient in ``grad_dtype`` and the all-gather of the BF16 parameters each move
    (world - 1) / world of the buffer per rank (ring or switch alike: every rank must ship every slice it does
    not own once), the norm exchange one double to every peer.  The BF16 + stochastic-rounding recipe
    communicates gradients in BF16 (Section 3), mixed precision in FP32: half the reduce-scatter bytes."""
    gsz = torch.empty(0, dtype=grad_dtype).element_size()
    share = (world_size - 1) / world_size if world_size > 0 else 0.0
    return {"reduce_scatter": int(n * gsz * share), "all_gather": int(n * 2 * share),
            "norm_exchange": 8 * max(0, world_size - 1), "grad_bytes_per_element": gsz}


def sharded_clipped_step(shard_p, shard_m, shard_v, full_grad, hp_kwargs: dict, seed: int, step: int, *, max_norm: float,
                         accum_scale: float = 1.0, tensor_id: int = 0, group=None, full_param_out=None, ops=None,
                         phase_hook=None, shard_grad_out=None):
    """One optimizer iteration with the state sharded over the ranks of ``group`` (ZeRO-1 shape):

        reduce-scatter(full_grad) -> grad_sqnorm -> rank-ordered global norm -> sr_clip_scale
        -> sr_adamw_step on this rank's slice with elem_offset = slice start -> all-gather(x)

    ``shard_p/m/v``: this rank's BF16 slice (length = partition(n)[rank][1]); ``full_grad``: this
    rank's full-length local gradient (FP32, or BF16 for the recipe's BF16 gradient communication;
    summed over ranks in that type by the reduce-scatter, the factor 1/world belongs in
    ``accum_scale``); ``full_param_out``: optional full-length BF16 buffer that receives every rank's
    updated slice; ``shard_grad_out``: optional buffer for the reduced slice (else allocated per call);
    ``phase_hook(name)``: called at the start of each phase and at the end ("reduce_scatter", "sqnorm",
    "norm_exchange", "clip_scale", "step", "all_gather", "end"), e.g. to record timing events.
    All slices must have equal length (n divisible by 8 * world), which is what the collectives need.  The collectives are torch.distributed calls
    (NCCL over NVLink on GPUs); every arithmetic step runs in the library's kernels.  ``ops`` lets a
    test substitute the four kernel calls; by default they are the CUDA binding's.
    Returns the global squared norm (one float64 tensor, identical on every rank).
    """
    world = dist.get_world_size(group)
    rank = dist.get_rank(group)
    n = full_grad.numel()
    if n % (8 * world) != 0:
        raise ValueError("buffer length must be a multiple of 8 * world size")
    per = n // world
    if not (shard_p.numel() == shard_m.numel() == shard_v.numel() == per):
        raise ValueError("shard length mismatch")
    if ops is None:
        from . import binding

        class ops:  # noqa: N801 - namespace of the four kernel calls
            @staticmethod
            def sqnorm(g, out):
                ws = torch.empty(max(1, binding.grad_sqnorm_workspace_bytes(g.numel()) // 8), dtype=torch.float64, device=g.device)
                binding.grad_sqnorm(g, out, ws)

            @staticmethod
            def clip_scale(total, accum, mx, out):
                binding.sr_clip_scale(total, accum, mx, out)

            @staticmethod
            def step(p, g, m, v, gscale_dev, offset):
                binding.sr_adamw_step(p, g, m, v, binding.hparams(**hp_kwargs, grad_scale_dev=gscale_dev), seed, step,
                                      tensor_id, offset)

    dev = full_grad.device
    mark = phase_hook if phase_hook is not None else (lambda name: None)
    shard_g = shard_grad_out if shard_grad_out is not None else torch.empty(per, dtype=full_grad.dtype, device=dev)
    if shard_g.numel() != per or shard_g.dtype != full_grad.dtype:
        raise ValueError("shard_grad_out must hold one slice of the gradient's type")
    mark("reduce_scatter")
    dist.reduce_scatter_tensor(shard_g, full_grad.contiguous(), op=dist.ReduceOp.SUM, group=group)
    mark("sqnorm")
    local = torch.zeros(1, dtype=torch.float64, device=dev)
    ops.sqnorm(shard_g, local)
    mark("norm_exchange")
    total = global_sqnorm(local, group)
    mark("clip_scale")
    gscale = torch.zeros(1, dtype=torch.float32, device=dev)
    ops.clip_scale(total, accum_scale, max_norm, gscale)
    mark("step")
    ops.step(shard_p, shard_g, shard_m, shard_v, gscale, rank * per)
    mark("all_gather")
    if full_param_out is not None:
        dist.all_gather_into_tensor(full_param_out, shard_p.contiguous(), group=group)
    mark("end")
    return total
