"""Plain-Python oracle for the group-schedule encoder.

TEST INFRASTRUCTURE ONLY.  It restates, as literally as possible, how a
synchronization-mode decision becomes the ordered list of worker groups that
one round of parameter updates walks through.  A schedule is returned as the
pair ``(group_offsets, group_members)`` of Python lists: group ``k`` consists of
``group_members[group_offsets[k]:group_offsets[k+1]]``.

Paper passages followed:
  * Section I: SSGD = one update from all N workers' gradients; ASGD = one
    update per worker's gradient, as they arrive.
  * Section I contribution (2), Section IV-B: static x-order = every update
    uses the gradients of x workers; dynamic x-order = every update uses the
    gradient reports of one cluster of workers with similar iteration times.
  * Section IV-C1 (text before Eq. 2): clusters are sorted in ascending order
    of the maximum iteration time inside the cluster.

Readings where the paper is silent:
  * x not dividing the number of arrived workers: the last group is smaller.
  * members inside a group are listed in ascending worker index when
    ``sort_members`` is set, otherwise in arrival order.
  * two clusters with the same maximum iteration time: the one holding the
    smaller worker index goes first.
  * a round may use fewer than all W workers; no worker may appear twice.
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

Schedule = Tuple[List[int], List[int]]


def is_valid(group_offsets: Sequence[int], group_members: Sequence[int], n_groups: int,
             W: int) -> bool:
    """True iff the CSR pair describes ``n_groups`` non-empty, disjoint groups of
    workers in ``[0, W)``."""
    if n_groups < 0 or W < 0:
        return False
    if n_groups == 0:
        return True
    if len(group_offsets) < n_groups + 1 or group_offsets[0] != 0:
        return False
    for k in range(n_groups):
        if group_offsets[k + 1] <= group_offsets[k]:
            return False
    total = group_offsets[n_groups]
    if total > len(group_members):
        return False
    seen = set()
    for j in range(total):
        w = group_members[j]
        if w < 0 or w >= W or w in seen:
            return False
        seen.add(w)
    return True


def _pack(groups: List[List[int]]) -> Schedule:
    offsets = [0]
    members: List[int] = []
    for g in groups:
        members.extend(g)
        offsets.append(len(members))
    return offsets, members


def static_x(arrival_order: Optional[Sequence[int]], W: int, x: int,
             sort_members: bool = False) -> Schedule:
    """Static x-order mode: consecutive runs of ``x`` workers in arrival order.

    ``arrival_order`` lists the workers whose gradients are used, earliest
    first (``None`` = ``0..W-1``).  ``x = W`` over all workers is SSGD, ``x = 1``
    is ASGD.
    """
    order = list(range(W)) if arrival_order is None else list(arrival_order)
    if x < 1:
        raise ValueError("x must be at least 1")
    if len(set(order)) != len(order) or any(w < 0 or w >= W for w in order):
        raise ValueError("arrival order must hold distinct workers in [0, W)")
    groups = []
    for start in range(0, len(order), x):
        g = order[start:start + x]
        groups.append(sorted(g) if sort_members else g)
    return _pack(groups)


def from_labels(group_of_worker: Sequence[int]) -> Schedule:
    """Groups from a per-worker label: group order = ascending label, members in
    ascending worker index; label ``-1`` = the worker takes no part."""
    if any(lab < -1 for lab in group_of_worker):
        raise ValueError("labels must be -1 or non-negative")
    labels = sorted({lab for lab in group_of_worker if lab >= 0})
    groups = [[w for w, lab in enumerate(group_of_worker) if lab == want] for want in labels]
    return _pack(groups)


def dynamic_x(iter_time: Sequence[float], cluster_of_worker: Sequence[int]) -> Schedule:
    """Dynamic x-order mode: one group per cluster, clusters c_1..c_Nc ascending
    in t_ci = the largest iteration time inside the cluster."""
    if len(iter_time) != len(cluster_of_worker):
        raise ValueError("need one iteration time and one cluster id per worker")
    if any(lab < -1 for lab in cluster_of_worker):
        raise ValueError("cluster ids must be -1 or non-negative")
    ids = sorted({c for c in cluster_of_worker if c >= 0})
    clusters = [[w for w, c in enumerate(cluster_of_worker) if c == want] for want in ids]
    keyed = []
    for members in clusters:
        t_c = max(iter_time[w] for w in members)
        keyed.append((t_c, members[0], members))
    keyed.sort(key=lambda item: (item[0], item[1]))
    return _pack([members for _, _, members in keyed])


def scaled_lrs(group_offsets: Sequence[int], n_groups: int, N: int, r_ssgd: float) -> List[float]:
    """Section IV-C1, learning-rate scaling: an update built from y gradient
    reports out of N workers runs at r_new = (y / N) * r_SSGD."""
    return [((group_offsets[k + 1] - group_offsets[k]) / N) * r_ssgd for k in range(n_groups)]
