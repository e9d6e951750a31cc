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


def shard_bounds(n: int, world: int, rank: int):
    """Contiguous equal shards; n must be a multiple of world (pad the flat buffer)."""
    if n % world:
        raise ValueError("buffer length must be a multiple of the world size")
    k = n // world
    return rank * k, (rank + 1) * k


def reduce_scatter_states(m: torch.Tensor, v: torch.Tensor, group=None):
    """Sums m and v over the ranks so that this rank's own shard holds the sum (in place);
    returns (lo, hi, world).  Backends without reduce-scatter fall back to an all-reduce."""
    world, rank = dist.get_world_size(group), dist.get_rank(group)
    lo, hi = shard_bounds(m.numel(), world, rank)
    for buf in (m, v):
        flat = buf.view(-1)
        try:
            dist.reduce_scatter_tensor(flat[lo:hi], flat, op=dist.ReduceOp.SUM, group=group)
        except (RuntimeError, NotImplementedError):
            dist.all_reduce(flat, op=dist.ReduceOp.SUM, group=group)
    return lo, hi, world


def reduce_scatter_apply_allgather(opt, w: torch.Tensor, m: torch.Tensor, v: torch.Tensor,
                                   lr: float, group=None) -> None:
    """End of a mini-batch with sharded optimizer states: reduce-scatter m, v; the owner
    updates its shard of w; shards of m, v owned by other ranks restart from zero; all-gather w."""
    lo, hi, world = reduce_scatter_states(m, v, group)
    wf, mf, vf = w.view(-1), m.view(-1), v.view(-1)
    opt.apply_sharded(wf[lo:hi], mf[lo:hi], vf[lo:hi], lr, world)
    mf[:lo].zero_()
    mf[hi:].zero_()
    vf[:lo].zero_()
    vf[hi:].zero_()
    try:
        dist.all_gather_into_tensor(wf, wf[lo:hi].clone(), group=group)
    except (RuntimeError, NotImplementedError):
        parts = [torch.empty_like(wf[lo:hi]) for _ in range(world)]
        dist.all_gather(parts, wf[lo:hi].clone(), group=group)
        wf.copy_(torch.cat(parts))


class PeerMappedStates:
    """w, m, v of one replica allocated in torch symmetric memory, so that every rank can
    address every other rank's buffers (NVLink peer access) and the whole end-of-mini-batch
    exchange is ONE kernel per rank (`AdamA.apply_sharded_peers`): no reduce-scatter, no
    all-gather.  The two barriers around it are the ordering the kernel asks of its caller.

    Written against torch.distributed._symmetric_memory; this repository's tests exercise the
    kernel with all ranks' buffers on one GPU (tests/test_gpu_ddp.py), not this allocation
    path on several GPUs.
    """

    def __init__(self, n: int, device, group=None):
        import torch.distributed._symmetric_memory as symm_mem
        self.group = group if group is not None else dist.group.WORLD
        self.world = dist.get_world_size(self.group)
        self.rank = dist.get_rank(self.group)
        if n % (4 * self.world):
            raise ValueError("n must be a multiple of 4 * world size (pad the flat buffer)")
        self.n = n
        self._bufs, self._handles = {}, {}
        for name in ("w", "m", "v"):
            t = symm_mem.empty(n, dtype=torch.float32, device=device)
            self._handles[name] = symm_mem.rendezvous(t, self.group)
            self._bufs[name] = t
        self.m.zero_()
        self.v.zero_()

    w = property(lambda self: self._bufs["w"])
    m = property(lambda self: self._bufs["m"])
    v = property(lambda self: self._bufs["v"])

    def exchange_and_apply(self, opt, lr: float) -> None:
        h = self._handles
        h["m"].barrier()          # every rank has finished folding into its m, v
        opt.apply_sharded_peers(list(h["w"].buffer_ptrs), list(h["m"].buffer_ptrs),
                                list(h["v"].buffer_ptrs), self.rank, self.n, lr)
        h["m"].barrier()          # every shard has been written everywhere
