"""One round over a communication tree across ranks.

Section IV-D2b: the workers of a job form a tree whose root is the parameter
server; every worker adds the partial sums it receives from its children to
its own gradient and forwards the result to its parent; the root updates the
parameters and sends them back down the tree.  Ranks 0 .. W-1 are the workers,
rank W is the root (it holds params and momentum and has no gradient).

This module only MOVES buffers (point-to-point sends and receives, always into
memory of the receiving rank's own device) and calls the two kernels that do
the arithmetic, ``star_group_reduce`` (own gradient + children's partial sums)
and ``star_group_update_from_sums`` (the root's sum over its children and the
update over N reports), through a backend object; it computes nothing itself.

Order of the additions: a worker's own gradient first, then its children's
partial sums in ascending worker index; the root adds its children's partial
sums in ascending worker index.  Partial sums travel as binary32: a worker first
widens its own gradient (exactly) when it has children, then adds.
"""
from __future__ import annotations

from typing import List, Sequence

import torch

from . import binding as B
from .all_reduce_round import CudaBackend


class TreePlan:
    """Who is whose child; identical on every rank."""

    def __init__(self, parent_of: Sequence[int]):
        self.W = len(parent_of)
        self.parent_of = [int(p) for p in parent_of]
        self.children: List[List[int]] = [[] for _ in range(self.W)]
        self.top: List[int] = []                       # the root's children, ascending
        for w, p in enumerate(self.parent_of):
            if p == w or p < -1 or p >= self.W:
                raise ValueError("bad parent for worker %d" % w)
            (self.top if p < 0 else self.children[p]).append(w)
        for w in range(self.W):                        # every worker must reach the root
            node, steps = w, 0
            while node != -1:
                node, steps = self.parent_of[node], steps + 1
                if steps > self.W:
                    raise ValueError("parent_of has a cycle")


class TreeRound:
    """Runs rounds on one rank of a world of W workers + 1 root (the last rank)."""

    def __init__(self, dist, rank: int, world: int, backend=None):
        self.dist, self.rank, self.W = dist, rank, world - 1
        self.backend = backend if backend is not None else CudaBackend()

    def run(self, grad, params: torch.Tensor, momentum, parent_of: Sequence[int], lr: float, mu: float,
            wd: float) -> TreePlan:
        """One round.  Workers pass their gradient and receive the updated ``params``
        (``momentum`` is not used on workers and may be None); the root passes
        ``grad=None`` and holds ``params`` and ``momentum``, updated in place."""
        dist, me, be = self.dist, self.rank, self.backend
        plan = TreePlan(parent_of)
        if plan.W != self.W:
            raise ValueError("need a parent for each of the %d workers" % self.W)
        n = params.numel()
        root = self.W
        mine = plan.top if me == root else plan.children[me]

        # bottom-up: receive the children's partial sums (binary32), add, forward
        received = [be.empty(n, torch.float32, params) for _ in mine]
        self._complete([dist.P2POp(dist.irecv, buf, c) for buf, c in zip(received, mine)])
        if me == root:
            be.update_from_sums(params, momentum, received, self.W, lr, mu, wd)
        else:
            up = root if plan.parent_of[me] < 0 else plan.parent_of[me]
            own = be.empty(n, torch.float32, params)
            be.reduce(own, [grad])                                     # exact widening to binary32
            if received:
                total = be.empty(n, torch.float32, params)
                be.reduce(total, [own] + received)
            else:
                total = own
            self._complete([dist.P2POp(dist.isend, total, up)])
        # top-down: parameters to the children
        if me != root:
            up = root if plan.parent_of[me] < 0 else plan.parent_of[me]
            self._complete([dist.P2POp(dist.irecv, params, up)])
        self._complete([dist.P2POp(dist.isend, params, c) for c in mine])
        return plan

    def _complete(self, ops) -> None:
        if ops:
            for req in self.dist.batch_isend_irecv(ops):
                req.wait()
