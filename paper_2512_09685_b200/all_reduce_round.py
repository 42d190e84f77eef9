"""One round of the all-reduce architecture across ranks (one rank = one worker).

Section IV-B, paragraph "All-reduce architecture", and Section IV-C1, Eq. 3:
x stragglers leave the ring; each reports its gradients to a parent in the
ring and gets parameters back from it; a parent adds the gradients of the
children that reported in time to its own; the ring sums its members'
aggregates; one update is made from the gradients of N - x + q workers.

This module only MOVES buffers (``torch.distributed`` point-to-point and
collective calls) and calls the two kernels that do the arithmetic,
``star_group_reduce`` and ``star_group_update_from_sums``, through a small
backend object; it computes nothing itself.  Every buffer a kernel sees is
memory of the rank's own device: a child's gradient is first received into a
local buffer, then reduced.

Summation order (fixed so that every rank ends with the same bits): a parent's
own gradient first, then its children in ascending worker index; the ring
members' aggregates in ascending worker index, for every element alike.  A
reducing collective is therefore NOT used for the ring sum (its order is the
library's choice and may depend on the element); the aggregates are exchanged
and summed locally by the update kernel:
  exchange="gather"   every ring member gathers all R aggregates and applies the
                      update to the whole tensor ((R - 1) n floats in per rank);
  exchange="scatter"  ring member j receives only its slice of every aggregate,
                      updates that slice of p and v, and the updated slices are
                      broadcast back: the volume of a ring all-reduce for the
                      aggregates ((R - 1) / R n floats in per rank) plus the
                      state slices out.
Both give bit-identical p and v on every ring member.
"""
from __future__ import annotations

from typing import Dict, List, Sequence

import torch

from . import binding as B


class CudaBackend:
    """The arithmetic of the round: the library's CUDA kernels on the current device."""

    def empty(self, n: int, dtype: torch.dtype, like: torch.Tensor) -> torch.Tensor:
        return torch.empty(n, dtype=dtype, device=like.device)

    def reduce(self, out: torch.Tensor, buffers: Sequence[torch.Tensor]) -> None:
        B.star_group_reduce(out, list(buffers), list(range(len(buffers))))

    def update_from_sums(self, params, momentum, sums, n_reports, lr, mu, wd) -> None:
        B.star_group_update_from_sums(params, momentum, list(sums), n_reports, lr, mu, wd)


class RoundPlan:
    """Who does what in a round; identical on every rank (host arithmetic only)."""

    def __init__(self, world: int, removed: Sequence[int], in_time: Sequence[int]):
        self.world = world
        self.removed = [int(c) for c in removed]
        self.in_time = sorted(int(c) for c in in_time)
        if not set(self.in_time) <= set(self.removed):
            raise ValueError("only removed workers can be children in time")
        self.parent_of = B.star_assign_parents(self.removed, world)       # -1 for ring members
        self.ring = [w for w in range(world) if self.parent_of[w] < 0]
        self.children: Dict[int, List[int]] = {r: [] for r in self.ring}   # in time, ascending
        for c in self.in_time:
            self.children[self.parent_of[c]].append(c)
        self.n_reports = len(self.ring) + len(self.in_time)                 # N - x + q of Eq. 3


def _bits(t: torch.Tensor) -> torch.Tensor:
    """bf16 travels as raw bytes (a type every transport moves; the bits arrive unchanged)."""
    return t.view(torch.uint8) if t.dtype == torch.bfloat16 else t


class AllReduceRound:
    """Runs rounds on one rank.  ``dist`` is ``torch.distributed`` (initialised);
    sub-groups for the rings are created on first use, by every rank in the
    same order, and cached."""

    def __init__(self, dist, rank: int, world: int, backend=None, exchange: str = "gather"):
        if exchange not in ("gather", "scatter"):
            raise ValueError(exchange)
        self.dist, self.rank, self.world = dist, rank, world
        self.backend = backend if backend is not None else CudaBackend()
        self.exchange = exchange
        self._groups: Dict[tuple, object] = {}

    def ring_group(self, ring: Sequence[int]):
        key = tuple(ring)
        if key not in self._groups:                      # collective: every rank calls it, member or not
            self._groups[key] = self.dist.new_group(ranks=list(ring)) if len(ring) < self.world else None
        return self._groups[key]

    def run(self, grad: torch.Tensor, params: torch.Tensor, momentum: torch.Tensor,
            removed: Sequence[int], in_time: Sequence[int], lr: float, mu: float, wd: float,
            hand_back_momentum: bool = True) -> RoundPlan:
        """One round, in place.  Ring members end with the updated ``params`` and
        ``momentum``; removed workers (in time or not) end with their parent's
        ``params`` and, unless ``hand_back_momentum`` is off (the same on every
        rank), its ``momentum`` too: the paper's children receive parameters;
        the optimizer state travels with them here so that a worker that rejoins
        the ring in a later round holds the state the ring holds."""
        dist, me, be = self.dist, self.rank, self.backend
        plan = RoundPlan(self.world, removed, in_time)
        n = params.numel()
        group = self.ring_group(plan.ring)
        i_am_in_ring = plan.parent_of[me] < 0

        # 1. children in time hand their gradient to their parent
        child_bufs: List[torch.Tensor] = []
        ops = []
        if i_am_in_ring:
            for c in plan.children[me]:
                buf = be.empty(n, grad.dtype, grad)
                child_bufs.append(buf)
                ops.append(dist.P2POp(dist.irecv, _bits(buf), c))
        elif me in plan.in_time:
            ops.append(dist.P2POp(dist.isend, _bits(grad), plan.parent_of[me]))
        self._complete(ops)

        if i_am_in_ring:
            # 2. own gradient + children, ascending
            aggregate = be.empty(n, torch.float32, params)
            be.reduce(aggregate, [grad] + child_bufs)
            # 3. exchange the aggregates, sum them in ring order inside the update kernel
            if self.exchange == "gather" or len(plan.ring) == 1:
                sums = [aggregate] if len(plan.ring) == 1 else self._gather(aggregate, plan.ring, group, be)
                be.update_from_sums(params, momentum, sums, plan.n_reports, lr, mu, wd)
            else:
                self._scatter_update(aggregate, params, momentum, plan, group, lr, mu, wd)

        # 4. parents hand the parameters to all their children, late ones included
        ops = []
        if i_am_in_ring:
            for c in plan.removed:
                if plan.parent_of[c] == me:
                    ops.append(dist.P2POp(dist.isend, params, c))
                    if hand_back_momentum:
                        ops.append(dist.P2POp(dist.isend, momentum, c))
        else:
            ops.append(dist.P2POp(dist.irecv, params, plan.parent_of[me]))
            if hand_back_momentum:
                ops.append(dist.P2POp(dist.irecv, momentum, plan.parent_of[me]))
        self._complete(ops)
        return plan

    # ------------------------------------------------------------------
    def _complete(self, ops) -> None:
        if ops:
            for req in self.dist.batch_isend_irecv(ops):
                req.wait()

    def _gather(self, aggregate, ring, group, be):
        sums = [be.empty(aggregate.numel(), torch.float32, aggregate) for _ in ring]
        self.dist.all_gather(sums, aggregate, group=group)
        return sums

    def _scatter_update(self, aggregate, params, momentum, plan: RoundPlan, group, lr, mu, wd) -> None:
        dist, be, ring = self.dist, self.backend, plan.ring
        R, n = len(ring), params.numel()
        slices = [B.star_shard_range(n, R, j, 16) for j in range(R)]
        mine = ring.index(self.rank)
        first, count = slices[mine]
        parts, ops = [], []
        for j, r in enumerate(ring):
            if j == mine:
                parts.append(aggregate[first:first + count])
                continue
            buf = be.empty(count, torch.float32, aggregate)
            parts.append(buf)
            if count:
                ops.append(dist.P2POp(dist.irecv, buf, r))
            f, c = slices[j]
            if c:
                ops.append(dist.P2POp(dist.isend, aggregate[f:f + c], r))
        self._complete(ops)
        if count:
            be.update_from_sums(params[first:first + count], momentum[first:first + count], parts, plan.n_reports,
                                lr, mu, wd)
        for j, r in enumerate(ring):                   # updated slices back to every ring member
            f, c = slices[j]
            if c:
                dist.broadcast(params[f:f + c], src=r, group=group)
                dist.broadcast(momentum[f:f + c], src=r, group=group)
