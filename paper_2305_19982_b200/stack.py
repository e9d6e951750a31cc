"""Stacks of linear layers driven through the AdamA library, back to front.

A `LinearStack` owns three flat fp32 device buffers (w, m, v) that hold every
layer's [d_in, d_out] matrix back to back; each layer is a view.  One mini-batch
follows Algorithm 2 of the AdamA paper: for every micro-batch the layers are
visited from the last to the first (the order in which backward produces their
gradients), each layer's (X, dY) pair is handed to the fused weight-gradient fold
(which also folds the layer's bias gradient when the stack has biases) and dropped at once, and after the last micro-batch every parameter is updated.
This module only sequences library calls and owns memory; all arithmetic is in
the CUDA kernels.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Callable, List, Sequence, Tuple

import torch

from .binding import AdamA


@dataclass(frozen=True)
class LayerSpec:
    name: str
    d_in: int
    d_out: int


class LinearStack:
    def __init__(self, layers: Sequence[LayerSpec], device="cuda", biases: bool = False):
        self.layers: List[LayerSpec] = list(layers)
        self.device = torch.device(device)
        self.biases = biases
        self.offsets: List[int] = []
        self.bias_offsets: List[int] = []
        total = 0
        for L in self.layers:
            self.offsets.append(total)
            total += L.d_in * L.d_out
            total = (total + 63) // 64 * 64  # keep every layer 256-byte aligned
            if biases:  # the layer's bias [d_out] follows its matrix
                self.bias_offsets.append(total)
                total = (total + L.d_out + 63) // 64 * 64
        self.numel = total
        self.w = torch.zeros(total, dtype=torch.float32, device=self.device)
        self.m = torch.zeros(total, dtype=torch.float32, device=self.device)
        self.v = torch.zeros(total, dtype=torch.float32, device=self.device)

    @property
    def n_params(self) -> int:
        return sum(L.d_in * L.d_out + (L.d_out if self.biases else 0) for L in self.layers)

    def bias_view(self, buf: torch.Tensor, j: int) -> torch.Tensor:
        o = self.bias_offsets[j]
        return buf[o:o + self.layers[j].d_out]

    def view(self, buf: torch.Tensor, j: int) -> torch.Tensor:
        L = self.layers[j]
        o = self.offsets[j]
        return buf[o:o + L.d_in * L.d_out].view(L.d_in, L.d_out)

    def flops_per_micro_batch(self, tokens: int) -> float:
        return sum(2.0 * tokens * L.d_in * L.d_out for L in self.layers)

    def fold_micro_batches(self, opt: AdamA, n_micro: int,
                           inputs: Callable[[int, int, LayerSpec], Tuple[torch.Tensor, torch.Tensor]],
                           layers_per_launch: int = 1) -> None:
        """The accumulation half of one mini-batch (Algorithm 2, inner loops): begin, then for
        every micro-batch every layer from the last to the first through the fused
        weight-gradient fold.  `inputs(micro, layer_index, spec)` returns (X, dY) for that
        (micro-batch, layer).  The weight gradient never exists in memory.  On return m, v
        hold m_t, v_t.

        layers_per_launch = 1: one call per layer, its (X, dY) released right after the call.
        layers_per_launch = k > 1: k consecutive layers (still back to front) go into one
        adama_linear_wgrad_fold_multi call, e.g. the four linears of a transformer block; their
        (X, dY) are released together after that call.  Same results, bit for bit."""
        opt.begin_minibatch(n_micro)
        for i in range(n_micro):
            pending = []
            for j in reversed(range(len(self.layers))):
                X, dY = inputs(i, j, self.layers[j])
                item = (X, dY, self.view(self.m, j), self.view(self.v, j))
                if self.biases:  # bias gradient (column sums of dY) in the same launch
                    item += (self.bias_view(self.m, j), self.bias_view(self.v, j))
                del X, dY
                if layers_per_launch <= 1:
                    opt.linear_wgrad_fold(*item)
                else:
                    pending.append(item)
                    if len(pending) == layers_per_launch:
                        opt.linear_wgrad_fold_multi(pending)
                        pending = []
                del item
            if pending:
                opt.linear_wgrad_fold_multi(pending)

    def apply(self, opt: AdamA, lr: float) -> None:
        """The update half (Algorithm 2, "Update"): one apply over the whole flat buffer (the
        padding between layers holds zeros); m, v leave it decayed for the next mini-batch."""
        opt.apply(self.w, self.m, self.v, lr)

    def minibatch(self, opt: AdamA, n_micro: int, lr: float,
                  inputs: Callable[[int, int, LayerSpec], Tuple[torch.Tensor, torch.Tensor]],
                  layers_per_launch: int = 1) -> None:
        """One whole mini-batch: fold_micro_batches, then apply."""
        self.fold_micro_batches(opt, n_micro, inputs, layers_per_launch)
        self.apply(opt, lr)


def gpt2xl_stack(blocks: int, device="cuda", biases: bool = False) -> LinearStack:
    h = 1600
    per_block = [("qkv", h, 3 * h), ("out_proj", h, h), ("fc1", h, 4 * h), ("fc2", 4 * h, h)]
    return LinearStack([LayerSpec(f"b{b}.{n}", di, do) for b in range(blocks)
                        for (n, di, do) in per_block], device, biases)


def llama7b_stack(blocks: int, device="cuda") -> LinearStack:
    h, f = 4096, 11008
    per_block = [("q", h, h), ("k", h, h), ("v", h, h), ("o", h, h),
                 ("gate", h, f), ("up", h, f), ("down", f, h)]
    return LinearStack([LayerSpec(f"b{b}.{n}", di, do) for b in range(blocks)
                        for (n, di, do) in per_block], device)
