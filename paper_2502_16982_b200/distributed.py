"""Owner-computes Muon over a data-parallel group (Sec. 2.3, Distributed Muon;
Algorithm 1).

Every rank holds the full weights of all Muon matrices.  Each matrix is owned
by one rank, which keeps its momentum and runs the step on it; the updated
weights are then all-gathered so that every rank ends with the same parameters
(Algorithm 1, last exchange).  Whole matrices are the unit of ownership, so the
"DP gather" of Algorithm 1 - assembling a full gradient matrix from partitions -
never arises: nothing is gathered inside the Newton-Schulz iteration.

Storage is laid out for collectives that need no staging copy.  Every shape
bucket of the planner (``muon_plan_buckets``) keeps its weights in ONE flat
tensor of ``world`` slots, slot r holding the matrices rank r owns
(``muon_partition_slots``), and its gradients in a second tensor of the same
layout.  The parameter all-gather of a bucket is then one in-place collective
(every rank's slot is written where it lives), and the gradient reduce-scatter
of Algorithm 1's first line one more (every owner receives the reduced
gradients of exactly its matrices).  The matrices the caller trains on are
views into these tensors (``weights`` / ``grads``).

Within a step the exchanges run bucket by bucket on a side stream: while the
compute stream is in bucket u's Newton-Schulz iteration, bucket u-1's weights go
out and bucket u+1's gradients come in, which is the overlap of gather and
computation, and of the optimizer's reduce-scatter with the parameter gather,
that Sec. 2.3 names.

This module is plumbing: ``torch.distributed`` for the collectives, the C-ABI
library (``muon_step_bucket``) for the arithmetic.  ``step_fn(mats, hp)``, with
``mats`` a list of (weight, grad, momentum), replaces the library call in tests
so that the collective logic can run on CPU ranks (gloo).
"""

from __future__ import annotations

from typing import Callable, Dict, List, Optional, Sequence, Tuple

import torch

from . import binding

_CODE = {torch.bfloat16: binding.MUON_DTYPE_BF16, torch.float32: binding.MUON_DTYPE_FP32}


class DistributedMuon:
    """``shapes``: list of (rows, cols, count, w_dtype, g_dtype), identical on
    every rank.  Allocates the flat per-bucket storage on ``device``; the
    matrices are ``self.weights[g][i]`` and ``self.grads[g][i]`` (views).
    Momentum is allocated for owned matrices only (the optimizer state is
    partitioned as in ZeRO-1, and is half of AdamW's)."""

    def __init__(self, shapes: Sequence[Tuple[int, int, int, torch.dtype, torch.dtype]], device, dist=None,
                 step_fn: Optional[Callable] = None):
        self.dist = dist
        self.rank = dist.get_rank() if dist is not None else 0
        self.world = dist.get_world_size() if dist is not None else 1
        self.device = torch.device(device)
        self.shapes = [tuple(s) for s in shapes]
        coded = [(r, c, n, _CODE[wd], _CODE[gd]) for (r, c, n, wd, gd) in self.shapes]
        self.unit_of, self.n_units = binding.muon_plan_buckets(coded)
        self.owners, self.pos, self.share, self.loads = binding.muon_partition_slots(coded, self.world)
        self.owned = [i for i, o in enumerate(self.owners) if o == self.rank]

        # flat storage: per unit [world * share, rows * cols] for weights and for gradients
        first_of_unit: Dict[int, int] = {}
        k = 0
        for gi, (r, c, n, wd, gd) in enumerate(self.shapes):
            first_of_unit.setdefault(self.unit_of[k], gi)
            k += n
        self.w_flat: List[torch.Tensor] = []
        self.g_flat: List[torch.Tensor] = []
        for u in range(self.n_units):
            r, c, n, wd, gd = self.shapes[first_of_unit[u]]
            slots = self.world * self.share[u]
            self.w_flat.append(torch.zeros((slots, r * c), dtype=wd, device=self.device))
            self.g_flat.append(torch.zeros((slots, r * c), dtype=gd, device=self.device))
        self.weights: List[List[torch.Tensor]] = []
        self.grads: List[List[torch.Tensor]] = []
        k = 0
        for (r, c, n, wd, gd) in self.shapes:
            ws, gs = [], []
            for j in range(n):
                u = self.unit_of[k + j]
                row = self.owners[k + j] * self.share[u] + self.pos[k + j]
                ws.append(self.w_flat[u][row].view(r, c))
                gs.append(self.g_flat[u][row].view(r, c))
            self.weights.append(ws)
            self.grads.append(gs)
            k += n

        # local groups: the owned matrices of every group, with fresh momentum
        self.local_groups = []
        local_flat = []
        k = 0
        for gi, (r, c, n, wd, gd) in enumerate(self.shapes):
            idx = [j for j in range(n) if self.owners[k + j] == self.rank]
            if idx:
                lw = [self.weights[gi][j] for j in idx]
                lg = [self.grads[gi][j] for j in idx]
                lm = [torch.zeros((r, c), dtype=torch.float32, device=self.device) for _ in idx]
                self.local_groups.append((lw, lg, lm))
                local_flat += [k + j for j in idx]
            k += n

        # this rank's bucket numbering (over its own matrices) against the global units
        self.local_bucket: List[Optional[int]] = [None] * self.n_units
        self.unit_mats: List[list] = [[] for _ in range(self.n_units)]
        if self.local_groups:
            lb, _ = binding.muon_plan_buckets(
                [(lw[0].shape[0], lw[0].shape[1], len(lw), _CODE[lw[0].dtype], _CODE[lg[0].dtype])
                 for lw, lg, _ in self.local_groups])
            triples = [t for lw, lg, lm in self.local_groups for t in zip(lw, lg, lm)]
            for p, flat in enumerate(local_flat):
                u = self.unit_of[flat]
                if self.local_bucket[u] is None:
                    self.local_bucket[u] = lb[p]
                elif self.local_bucket[u] != lb[p]:
                    raise RuntimeError("local and global bucket numbering disagree")
                self.unit_mats[u].append(triples[p])

        self._step_fn = step_fn
        self._ctx = None
        if step_fn is None and self.local_groups:
            self._ctx = binding.MuonContext(self.local_groups)
        self._cuda = self.device.type == "cuda"
        self._comm = torch.cuda.Stream(device=self.device) if (self._cuda and self.world > 1) else None
        # collectives on tensors: NCCL has them for CUDA tensors, gloo for CPU tensors; with gloo on
        # CUDA tensors (tests on one GPU) only broadcast and all-reduce exist, which serve as well
        backend = dist.get_backend() if dist is not None else None
        self._tensor_collectives = not (self._cuda and backend == "gloo")
        self.gather_bytes_per_rank = sum(
            (self.world - 1) * self.share[u] * self.w_flat[u].shape[1] * self.w_flat[u].element_size()
            for u in range(self.n_units)) if self.world > 1 else 0

    # -- the exchanges (in place on the flat storage) -------------------------
    def _slot(self, flat: torch.Tensor, u: int, r: int) -> torch.Tensor:
        return flat[r * self.share[u]:(r + 1) * self.share[u]]

    def _all_gather_unit(self, u: int) -> None:
        """Algorithm 1, last exchange: every rank's slot of bucket u to all ranks."""
        flat = self.w_flat[u]
        if self._tensor_collectives:
            self.dist.all_gather_into_tensor(flat, self._slot(flat, u, self.rank))
        else:
            for r in range(self.world):
                self.dist.broadcast(self._slot(flat, u, r), src=r)

    def _reduce_scatter_unit(self, u: int) -> None:
        """Algorithm 1, first line: the sum over ranks of bucket u's gradients,
        each owner receiving its own slot."""
        flat = self.g_flat[u]
        if self._tensor_collectives:
            self.dist.reduce_scatter_tensor(self._slot(flat, u, self.rank), flat)
        else:
            self.dist.all_reduce(flat)

    # -- one optimizer step ------------------------------------------------------
    def step(self, hp, reduce_grads: bool = False, timing: Optional[dict] = None) -> None:
        """One Muon step on the owned matrices and the exchange of the results.

        ``reduce_grads``: the gradient tensors hold this rank's local gradients
        and are summed over the ranks first (reduce-scatter); otherwise they are
        taken as already reduced on the owner.  ``timing``: a dict that receives
        CUDA events (``start``, ``compute_end``, ``end`` and the pairs
        ``exchanges``) for the benchmark."""
        if self.world == 1:
            if timing is not None and self._cuda:
                timing["start"] = self._mark(torch.cuda.current_stream(self.device))
                timing["exchanges"] = []
            for u in range(self.n_units):
                self._compute_unit(u, hp)
            if timing is not None and self._cuda:
                timing["compute_end"] = timing["end"] = self._mark(torch.cuda.current_stream(self.device))
            return
        if self._comm is None:  # CPU ranks: everything in program order
            for u in range(self.n_units):
                if reduce_grads:
                    self._reduce_scatter_unit(u)
                self._compute_unit(u, hp)
                self._all_gather_unit(u)
            return
        main = torch.cuda.current_stream(self.device)
        comm = self._comm
        mark = (lambda s: self._mark(s)) if timing is not None else (lambda s: None)
        if timing is not None:
            timing["start"] = self._mark(main)
            timing["exchanges"] = []
        comm.wait_stream(main)  # gradients and weights are final once the compute stream reaches this point
        grads_ready: List[Optional[torch.cuda.Event]] = [None] * self.n_units

        def exchange(fn, u):
            with torch.cuda.stream(comm):
                t0 = mark(comm)
                fn(u)
                t1 = mark(comm)
                if timing is not None:
                    timing["exchanges"].append((t0, t1))

        def reduce(u):
            exchange(self._reduce_scatter_unit, u)
            ev = torch.cuda.Event()
            ev.record(comm)
            grads_ready[u] = ev

        if reduce_grads:
            reduce(0)
        for u in range(self.n_units):
            # the next bucket's gradients are queued before this bucket's gather, which has to wait
            # for the compute stream
            if reduce_grads and u + 1 < self.n_units:
                reduce(u + 1)
            if grads_ready[u] is not None:
                main.wait_event(grads_ready[u])
            self._compute_unit(u, hp)
            done = torch.cuda.Event()
            done.record(main)
            comm.wait_event(done)
            exchange(self._all_gather_unit, u)
        if timing is not None:
            timing["compute_end"] = self._mark(main)
        main.wait_stream(comm)
        if timing is not None:
            timing["end"] = self._mark(main)

    @staticmethod
    def _mark(stream):
        ev = torch.cuda.Event(enable_timing=True)
        ev.record(stream)
        return ev

    def _compute_unit(self, u: int, hp) -> None:
        lb = self.local_bucket[u]
        if lb is None:
            return
        if self._step_fn is not None:
            self._step_fn(self.unit_mats[u], hp)
        else:
            self._ctx.muon_step_bucket(hp, lb)

    def all_gather_weights(self) -> None:
        """Every rank ends with every owner's current weights (all buckets)."""
        if self.world == 1:
            return
        for u in range(self.n_units):
            self._all_gather_unit(u)

    def status(self):
        """(status code, matrix index) of this rank's context (synchronises)."""
        return self._ctx.muon_status() if self._ctx is not None else (0, -1)

    def close(self) -> None:
        if self._ctx is not None:
            self._ctx.muon_destroy()
            self._ctx = None
