"""Owner-computes Muon over a data-parallel group (Sec. 2.3, Distributed Muon).

Every rank holds the full weights and the reduced gradients of all Muon
matrices.  Each matrix is owned by one rank (``muon_partition``: balanced by
Newton-Schulz work); the owner keeps its momentum, runs the step on it, and the
updated weights are then all-gathered so every rank ends with the same
parameters.  Because whole matrices are the unit of ownership, nothing is
gathered inside the Newton-Schulz iteration; the only collective is the
parameter all-gather that ZeRO-1 AdamW performs too.

The gather runs shape bucket by shape bucket (``muon_plan_buckets`` over the
full parameter list, so every rank sees the same buckets): as soon as a rank's
share of one bucket is stepped, that bucket's weights go out on a side stream
while the compute stream carries on with the next bucket's iteration, which is
the overlap of gather and computation Sec. 2.3 asks for.  The side stream is
in order, so one staging buffer serves all buckets.

This module is plumbing: torch.distributed for the collective, the C-ABI
library (``muon_step_bucket``) for the arithmetic.  ``step_fn(mats, hp)``, with
``mats`` a list of (weight, grad, momentum), replaces the library call in tests
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

        # units of the gather: the planner's buckets over ALL matrices
        dt = binding._dtype_code
        self.unit_of, self.n_units = binding.muon_plan_buckets(
            [(ws[0].shape[0], ws[0].shape[1], len(ws), dt(ws[0]), dt(gs[0])) for ws, gs in groups])

        # local groups: the owned matrices of every original group, with fresh momentum
        self.local_groups = []
        local_flat = []  # flat index of every local matrix, local groups in order
        k = 0
        for ws, gs in groups:
            idx = [j for j in range(len(ws)) if self.owners[k + j] == self.rank]
            if idx:
                lw, lg = [ws[j] for j in idx], [gs[j] for j in idx]
                lm = [torch.zeros(w.shape, dtype=torch.float32, device=w.device) for w in lw]
                self.local_groups.append((lw, lg, lm))
                local_flat += [k + j for j in idx]
            k += len(ws)

        # this rank's bucket numbering (over its own matrices) against the global units
        self.local_bucket: List[Optional[int]] = [None] * self.n_units
        self.unit_mats: List[list] = [[] for _ in range(self.n_units)]
        if self.local_groups:
            lb, _ = binding.muon_plan_buckets(
                [(lw[0].shape[0], lw[0].shape[1], len(lw), dt(lw[0]), dt(lg[0])) for lw, lg, _ in self.local_groups])
            triples = [t for lw, lg, lm in self.local_groups for t in zip(lw, lg, lm)]
            for pos, flat in enumerate(local_flat):
                u = self.unit_of[flat]
                if self.local_bucket[u] is None:
                    self.local_bucket[u] = lb[pos]
                elif self.local_bucket[u] != lb[pos]:
                    raise RuntimeError("local and global bucket numbering disagree")
                self.unit_mats[u].append(triples[pos])

        self._step_fn = step_fn
        self._ctx = None
        if step_fn is None and self.local_groups:
            self._ctx = binding.MuonContext(self.local_groups)

        # gather plan per unit: every rank sends its owned weights of the unit
        # back to back, padded to the unit's largest share
        self.unit_members: List[List[int]] = [[] for _ in range(self.n_units)]
        for i, u in enumerate(self.unit_of):
            self.unit_members[u].append(i)
        self.unit_pad = []
        for u in range(self.n_units):
            share = [0] * self.world
            for i in self.unit_members[u]:
                share[self.owners[i]] += self.flat_w[i].numel()
            self.unit_pad.append(max(share))
        ref = self.flat_w[0]
        self._cuda = ref.is_cuda
        self._stage = None
        self._comm = None
        if self.world > 1:
            most = max(self.unit_pad[u] * self.flat_w[self.unit_members[u][0]].element_size()
                       for u in range(self.n_units))
            # [send | recv of rank 0 | ... | recv of rank world-1], whole elements of any dtype
            self._stage = torch.empty((self.world + 1) * ((most + 15) // 16 * 16), dtype=torch.uint8,
                                      device=ref.device)
            if self._cuda:
                self._comm = torch.cuda.Stream(device=ref.device)

    # -- one optimizer step ------------------------------------------------
    def step(self, hp) -> None:
        for u in range(self.n_units):
            lb = self.local_bucket[u]
            if lb is not None:
                if self._step_fn is not None:
                    self._step_fn(self.unit_mats[u], hp)
                else:
                    self._ctx.muon_step_bucket(hp, lb)
            self._gather_unit(u)
        if self._comm is not None:
            torch.cuda.current_stream(self.flat_w[0].device).wait_stream(self._comm)

    def all_gather_weights(self) -> None:
        """Every rank ends with every owner's current weights (all units)."""
        for u in range(self.n_units):
            self._gather_unit(u)
        if self._comm is not None:
            torch.cuda.current_stream(self.flat_w[0].device).wait_stream(self._comm)

    def _gather_unit(self, u: int) -> None:
        if self.world == 1 or self.unit_pad[u] == 0:
            return
        if self._comm is None:
            self._gather_unit_on_current_stream(u)
            return
        # weights of unit u are final once the compute stream reaches this point
        self._comm.wait_stream(torch.cuda.current_stream(self.flat_w[0].device))
        with torch.cuda.stream(self._comm):
            self._gather_unit_on_current_stream(u)

    def _gather_unit_on_current_stream(self, u: int) -> None:
        members = self.unit_members[u]
        w0 = self.flat_w[members[0]]
        pad = self.unit_pad[u]
        nbytes = pad * w0.element_size()
        lane = self._stage.numel() // (self.world + 1)
        send = self._stage[:nbytes].view(w0.dtype)
        recv_all = self._stage[lane:].view(self.world, lane)[:, :nbytes]
        recv = [recv_all[r].view(w0.dtype) for r in range(self.world)]
        off = 0
        for i in members:
            if self.owners[i] == self.rank:
                w = self.flat_w[i]
                send[off:off + w.numel()].view(w.shape).copy_(w)
                off += w.numel()
        if off < pad:
            send[off:].zero_()
        self.dist.all_gather(recv, send)
        offs = [0] * self.world
        for i in members:
            o = self.owners[i]
            w = self.flat_w[i]
            if o != self.rank:
                w.copy_(recv[o][offs[o]:offs[o] + w.numel()].view(w.shape))
            offs[o] += w.numel()

    def close(self) -> None:
        if self._ctx is not None:
            self._ctx.muon_destroy()
            self._ctx = None
