"""Plain oracle of one round over a communication tree.

TEST INFRASTRUCTURE ONLY.  Section IV-D2b (paragraph on amortizing the
communication overhead): the workers of a job are arranged in a tree whose
root is the parameter server (in the all-reduce architecture: a parent);
workers with longer communication latency sit in lower layers; every worker
adds the gradients it receives from its children to its own and forwards the
result upward; the root updates the parameters, which travel back top-down.
The tree is rebuilt before every iteration.

The round, in the paper's order:
  1. every worker w forms  s_w = g_w + s_c1 + s_c2 + ...   (its children c1 < c2 < ...),
     leaves first, and forwards s_w to its parent;
  2. the root forms         S = s_r1 + s_r2 + ...            (its children r1 < r2 < ...);
  3. the root applies ONE update with the mean  S / N  over the N workers:
         d = fma(wd, p, gbar) ; v = fma(mu, v, d) ; p = fma(-lr, v, p);
  4. the parameters go back down the tree.

Readings where the paper is silent (it gives neither a fan-out, nor a rule for
filling the layers beyond "longer latency lower", nor a summation order):
  * shape: a k-ary tree filled layer by layer in ascending latency (ties: smaller
    worker index first): the k quickest workers are the root's children, the
    next k the children of the quickest one, and so on;
  * a worker's own gradient comes first, then its children's partial sums in
    ascending worker index; each addition is one binary32 operation; partial
    sums travel as binary32 (a bf16 gradient is widened exactly before it is
    added);
  * the root adds its children's partial sums in ascending worker index;
  * every worker reports in such a round, so the mean divides by N, and momentum
    and weight decay apply once (the round is SSGD carried by a tree).
The additions and the update are those of star_oracle.c (oracle_group_reduce_f32,
oracle_update_from_sums_f32); this module only composes them.
"""
from __future__ import annotations

from typing import Dict, List, Sequence

import numpy as np

from . import star_oracle as O


def build_tree(latency: Sequence[float], fanout: int) -> List[int]:
    """parent_of[w] for every worker; -1 = child of the root."""
    if fanout < 1:
        raise ValueError("fanout must be at least 1")
    order = sorted(range(len(latency)), key=lambda w: (latency[w], w))
    parent_of = [-1] * len(latency)
    for i, w in enumerate(order):
        if i >= fanout:
            parent_of[w] = order[(i - fanout) // fanout]
    return parent_of


def children_lists(parent_of: Sequence[int]) -> Dict[int, List[int]]:
    """node -> its children ascending; key -1 is the root."""
    out: Dict[int, List[int]] = {-1: []}
    for w in range(len(parent_of)):
        out.setdefault(w, [])
    for w, p in enumerate(parent_of):
        out[int(p)].append(w)
    return out


def partial_sums_f32(grads, parent_of: Sequence[int]) -> List[np.ndarray]:
    """s_w for every worker (float32 arrays): what w forwards to its parent."""
    kids = children_lists(parent_of)
    W = len(parent_of)
    done: Dict[int, np.ndarray] = {}

    def visit(w: int, depth: int) -> np.ndarray:
        if depth > W:
            raise ValueError("parent_of has a cycle")
        if w not in done:
            own = O.group_reduce_f32([grads[w]], [0])                         # exact widening
            parts = [own] + [visit(c, depth + 1) for c in kids[w]]
            done[w] = O.group_reduce_f32(parts, list(range(len(parts))))      # left to right
        return done[w]

    return [visit(w, 0) for w in range(W)]


def tree_round_f32(params: np.ndarray, momentum: np.ndarray, grads, parent_of: Sequence[int], lr, mu, wd):
    """One round, in place on ``params`` / ``momentum`` (the root's copy, which
    every worker holds after step 4).  ``grads[w]``: float32 or uint16 (bf16
    bits) array of worker w.  Returns the partial sums per worker."""
    sums = partial_sums_f32(grads, parent_of)
    top = children_lists(parent_of)[-1]
    if not top:
        raise ValueError("the root has no children")
    O.update_from_sums_f32(params, momentum, [sums[w] for w in top], len(parent_of), lr, mu, wd)   # steps 2, 3
    return sums
