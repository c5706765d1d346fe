"""Owner-computes Muon over a data-parallel group (Sec. 2.3, Distributed Muon).

Every rank holds the full weights and the reduced gradients of all Muon
matrices.  Each matrix is owned by one rank (``muon_partition``: balanced by
Newton-Schulz work); the owner keeps its momentum, runs the step on it, and the
updated weights are then all-gathered so every rank ends with the same
parameters.  Because whole matrices are the unit of ownership, nothing is
gathered inside the Newton-Schulz iteration; the only collective is the
parameter all-gather that ZeRO-1 AdamW performs too.

This module is plumbing: torch.distributed for the collective, the C-ABI
library (through ``step_fn``) for the arithmetic.  ``step_fn`` defaults to a
:class:`~paper_2502_16982_b200.binding.MuonContext` step; tests pass a stand-in
so the collective logic can run on CPU ranks (gloo).
"""

from __future__ import annotations

from typing import Callable, List, Optional, Sequence

import torch

from . import binding


class DistributedMuon:
    """``groups``: list of (weights, grads) with lists of equal-shaped 2-D
    tensors, identical on every rank.  Momentum is allocated for owned
    matrices only (half of AdamW's optimizer state, partitioned as in ZeRO-1)."""

    def __init__(self, groups: Sequence[Sequence[Sequence[torch.Tensor]]], dist=None,
                 step_fn: Optional[Callable] = None):
        self.dist = dist
        self.rank = dist.get_rank() if dist is not None else 0
        self.world = dist.get_world_size() if dist is not None else 1
        shapes = [(ws[0].shape[0], ws[0].shape[1], len(ws)) for ws, _ in groups]
        self.owners, self.loads = binding.muon_partition(shapes, self.world)
        self.flat_w: List[torch.Tensor] = [w for ws, _ in groups for w in ws]
        self.owned = [i for i, o in enumerate(self.owners) if o == self.rank]
        # local groups: the owned matrices of every original group, with fresh momentum
        self.local_groups = []
        k = 0
        for ws, gs in groups:
            idx = [j for j in range(len(ws)) if self.owners[k + j] == self.rank]
            k += len(ws)
            if idx:
                lw, lg = [ws[j] for j in idx], [gs[j] for j in idx]
                lm = [torch.zeros(w.shape, dtype=torch.float32, device=w.device) for w in lw]
                self.local_groups.append((lw, lg, lm))
        self._step_fn = step_fn
        self._ctx = None
        if step_fn is None and self.local_groups:
            self._ctx = binding.MuonContext(self.local_groups)
        # gather plan: every rank sends its owned weights back to back, padded to the largest share
        self.counts = [sum(self.flat_w[i].numel() for i, o in enumerate(self.owners) if o == r)
                       for r in range(self.world)]
        self.pad = max(self.counts) if self.counts else 0

    def step(self, hp) -> None:
        if self._step_fn is not None:
            self._step_fn(self.local_groups, hp)
        elif self._ctx is not None:
            self._ctx.muon_step(hp)
        self.all_gather_weights()

    def all_gather_weights(self) -> None:
        """Every rank ends with every owner's updated weights."""
        if self.dist is None or self.world == 1 or self.pad == 0:
            return
        ref = self.flat_w[0]
        send = torch.zeros(self.pad, dtype=ref.dtype, device=ref.device)
        off = 0
        for i in self.owned:
            w = self.flat_w[i]
            send[off:off + w.numel()].copy_(w.reshape(-1))
            off += w.numel()
        recv = [torch.empty(self.pad, dtype=ref.dtype, device=ref.device) for _ in range(self.world)]
        self.dist.all_gather(recv, send)
        offs = [0] * self.world
        for i, o in enumerate(self.owners):
            w = self.flat_w[i]
            if o != self.rank:
                w.copy_(recv[o][offs[o]:offs[o] + w.numel()].view(w.shape))
            offs[o] += w.numel()

    def close(self) -> None:
        if self._ctx is not None:
            self._ctx.muon_destroy()
            self._ctx = None
