"""Plain oracle of one round of the all-reduce architecture.

TEST INFRASTRUCTURE ONLY.  Section IV-B (paragraph "All-reduce architecture"):
x of the stragglers are taken out of the ring; each reports its gradients to a
non-straggler parent and receives parameters from it; a parent waits t_w after
its own computation, then aggregates its own gradients and those of its
children and hands the aggregate to the ring.  Section IV-C1, Eq. 3 counts the
batch of such a round as (N - x + q) M / N: the ring members plus the q
children whose reports were in before the wait ran out.

The round, in the paper's order:
  1. every removed worker that is in time hands its gradient to its parent;
  2. every ring member forms  a_r = g_r + g_c1 + g_c2 + ...  (children c1 < c2 < ...);
  3. the ring all-reduces:    S = a_r0 + a_r1 + ...           (ring order);
  4. every ring member applies ONE update with the mean  S / (N - x + q):
         d = fma(wd, p, gbar) ; v = fma(mu, v, d) ; p = fma(-lr, v, p);
  5. every child receives its parent's parameters.

Readings where the paper is silent (it fixes no summation order and does not
say how parents are picked beyond "a non-straggler that has high bandwidth"):
  * a parent's own gradient comes first, then its children in ascending worker
    index; each addition is one binary32 operation;
  * the ring is the remaining workers in ascending worker index and its sum
    runs left to right in that order, for every element alike (a transport
    whose order depends on the element, such as a chunked ring, would give
    another rounding);
  * the mean divides by the number of gradient reports, not of ring members;
  * momentum and weight decay apply once per round, as in SSGD;
  * parents: behind a non-blocking switch every ring member is equally near, so
    the removed workers are dealt round-robin (slowest first) over the ring in
    ascending index, which also balances the number of children per parent
    (Section IV-D2a).
The arithmetic of steps 2-4 is in star_oracle.c (oracle_group_reduce_f32,
oracle_update_from_sums_f32); this module only composes them.
"""
from __future__ import annotations

from typing import Dict, List, Sequence

import numpy as np

from . import star_oracle as O


def assign_parents(removed: Sequence[int], ring: Sequence[int]) -> Dict[int, int]:
    """child -> parent: the j-th removed worker (as listed, slowest first) goes
    to ring member j mod R of the ring in ascending index."""
    order = sorted(ring)
    return {int(c): int(order[j % len(order)]) for j, c in enumerate(removed)}


def children_of(parent_of: Dict[int, int], in_time: Sequence[int]) -> Dict[int, List[int]]:
    """parent -> its children whose reports count, ascending."""
    out: Dict[int, List[int]] = {}
    for c in sorted(in_time):
        out.setdefault(parent_of[c], []).append(int(c))
    return out


def all_reduce_round_f32(params: np.ndarray, momentum: np.ndarray, grads, ring: Sequence[int],
                         parent_of: Dict[int, int], in_time: Sequence[int], lr, mu, wd):
    """One round, in place on ``params`` / ``momentum`` (the copy every ring
    member and, after step 5, every child holds).  ``grads[w]``: float32 or
    uint16 (bf16 bits) array of worker w, None for workers that contribute
    nothing.  Returns (aggregates per ring member in ring order, n_reports)."""
    ring = sorted(int(r) for r in ring)
    kids = children_of(parent_of, in_time)
    aggregates = [O.group_reduce_f32(grads, [r] + kids.get(r, [])) for r in ring]        # step 2
    n_reports = len(ring) + len(in_time)
    O.update_from_sums_f32(params, momentum, aggregates, n_reports, lr, mu, wd)          # steps 3, 4
    return aggregates, n_reports
