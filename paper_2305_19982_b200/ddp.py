"""Data-parallel AdamA (Section 3.3 of the paper): the optimizer STATES are all-reduced once
per mini-batch instead of the gradients once per micro-batch.

Each rank folds its own micro-batches into its own m and v (which start the mini-batch as
beta1*m_t and R*beta2*v_t); at the end of the mini-batch `allreduce_states` sums m and v over
the ranks with torch.distributed (NCCL on GPUs) and `AdamA.apply_allreduced` turns the sums
into the update (division by R and R^2 folded into the kernel's constants).  This module
only sequences the collective and the library call.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def allreduce_states(m: torch.Tensor, v: torch.Tensor, group=None) -> int:
    """Sums m and v over the ranks of `group`, in place; returns the group's size."""
    dist.all_reduce(m, op=dist.ReduceOp.SUM, group=group)
    dist.all_reduce(v, op=dist.ReduceOp.SUM, group=group)
    return dist.get_world_size(group)


def allreduce_and_apply(opt, w: torch.Tensor, m: torch.Tensor, v: torch.Tensor, lr: float,
                        group=None) -> None:
    """End of a mini-batch on every rank: one state all-reduce, then the fused update."""
    world = allreduce_states(m, v, group)
    opt.apply_allreduced(w, m, v, lr, world)
