"""Plain-Python oracle for the host-side mode decision that feeds the schedule.

TEST INFRASTRUCTURE ONLY.  It restates, for N workers with predicted iteration
times t_1..t_N:

  * Section IV-B: the dynamic x-order mode clusters workers with similar
    predicted iteration times by agglomerative hierarchical clustering.
  * Section IV-C1, Eq. 1:  T_x = (1 + phi_k / (x M / N)) * t_x   for the static
    x-order modes (x = 1 is ASGD, x = N is SSGD),
  * Section IV-C1, Eq. 2:  T_d = 1 / sum_i 1 / ((1 + phi_k / (n_ci M / N)) * t_ci)
    for the dynamic mode with clusters c_1..c_Nc of n_ci workers whose slowest
    member takes t_ci,
  * and the choice of the mode with the smallest time.

phi_k is the pre-conditioned gradient noise scale of the current update and M
the total batch size; both are inputs here.

Readings where the paper is silent:
  * linkage: average linkage (mean pairwise |t_a - t_b|); ties between equally
    close pairs go to the pair whose clusters hold the smallest worker indices.
  * stopping: merge while more than `n_clusters` clusters remain (if given) and
    the closest pair is no farther apart than `max_distance` (if given).
  * t_x, "the expected time needed for one parameter update" of a static x-order
    mode: the time until x gradient reports are in when all workers start
    together, i.e. the x-th smallest predicted iteration time (t_1 = fastest
    worker for ASGD, t_N = slowest worker for SSGD).  This is the reading under
    which the model behaves as Section IV-B describes: without stragglers a
    higher order wins, a straggler inflates t_N and pushes the choice down.
  * ties between modes: the larger x wins (more synchronous), static before
    dynamic.
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple


def agglomerative_clusters(iter_time: Sequence[float], n_clusters: Optional[int] = None,
                           max_distance: Optional[float] = None) -> List[int]:
    """Cluster label per worker; labels numbered by each cluster's smallest
    worker index in ascending order."""
    N = len(iter_time)
    clusters = [[w] for w in range(N)]
    want = 1 if n_clusters is None else max(1, n_clusters)
    while len(clusters) > want:
        best = None
        for a in range(len(clusters)):
            for b in range(a + 1, len(clusters)):
                pairs = [(i, j) for i in clusters[a] for j in clusters[b]]
                dist = sum(abs(iter_time[i] - iter_time[j]) for i, j in pairs) / len(pairs)
                key = (dist, min(clusters[a]), min(clusters[b]))
                if best is None or key < best[0]:
                    best = (key, a, b)
        (dist, _, _), a, b = best
        if max_distance is not None and dist > max_distance:
            break
        clusters[a] = sorted(clusters[a] + clusters[b])
        del clusters[b]
        clusters.sort(key=min)
    labels = [0] * N
    for label, members in enumerate(sorted(clusters, key=min)):
        for w in members:
            labels[w] = label
    return labels


def time_static_x(iter_time: Sequence[float], x: int, phi: float, M: float) -> float:
    """Eq. 1."""
    N = len(iter_time)
    t_x = sorted(iter_time)[x - 1]
    return (1.0 + phi / (x * M / N)) * t_x


def time_dynamic(iter_time: Sequence[float], labels: Sequence[int], phi: float, M: float) -> float:
    """Eq. 2."""
    N = len(iter_time)
    total = 0.0
    for c in sorted(set(labels)):
        members = [w for w in range(N) if labels[w] == c]
        n_c = len(members)
        t_c = max(iter_time[w] for w in members)
        total += 1.0 / ((1.0 + phi / (n_c * M / N)) * t_c)
    return 1.0 / total


def choose_mode(iter_time: Sequence[float], labels: Sequence[int], phi: float,
                M: float) -> Tuple[int, float]:
    """(x, T): x in 1..N for the static x-order mode with the smallest time, or
    x = 0 if the dynamic mode with the given clusters beats every static one."""
    N = len(iter_time)
    best_x, best_T = N, time_static_x(iter_time, N, phi, M)
    for x in range(N - 1, 0, -1):
        T = time_static_x(iter_time, x, phi, M)
        if T < best_T:
            best_x, best_T = x, T
    T_d = time_dynamic(iter_time, labels, phi, M)
    if T_d < best_T:
        best_x, best_T = 0, T_d
    return best_x, best_T


# ---------------------------------------------------------------------------
# All-reduce architecture (Section IV-B "All-reduce architecture", Section
# IV-C1 Eq. 3): remove x of the X stragglers from the ring, attach each to a
# parent; parents wait t_w after the ring's slowest member is done and add the
# gradients of the children that have reported by then.
#
#   Section II:  d_i = (T_i - min T) / min T;  worker i is a straggler iff d_i > 20 %.
#   Eq. 3:       T_a = (1 + phi_k / ((N - x + q) M / N)) * (t_ring + t_w)
#
# Readings where the paper is silent or loose:
#   * which x stragglers are removed: the x slowest (ties: larger index first).
#   * q, which the paper describes as the number of removed stragglers whose
#     new iteration time does not exceed t_w: a removed worker w has a predicted
#     iteration time as a child, child_time[w]; t_w is a wait that starts when
#     the ring's slowest member is done, so w counts iff child_time[w] - t_ring
#     <= t_w, i.e. its report is in before its parent stops waiting.  (Read
#     literally, child_time[w] <= t_w, a child would have to finish within the
#     wait alone; time_all_reduce(..., literal=True) evaluates that reading so
#     that a test can show where the two part.)
#   * range of t_w: 0 <= t_w <= t_w_max.  Only t_w = 0 and the values at which
#     one more child makes it, child_time[w] - t_ring, can be optimal.
#   * ties: fewer removed workers, then the shorter wait.
# The gradients that enter the update are those of the ring members and of the
# q children in time: on a parameter server holding all buffers this is ONE
# group of N - x + q workers (a partial cover of the N workers).
# ---------------------------------------------------------------------------
def deviation_ratios(iter_time: Sequence[float]) -> List[float]:
    fastest = min(iter_time)
    return [(t - fastest) / fastest for t in iter_time]


def stragglers(iter_time: Sequence[float], threshold: float = 0.2) -> List[int]:
    return [w for w, d in enumerate(deviation_ratios(iter_time)) if d > threshold]


def time_all_reduce(iter_time: Sequence[float], child_time: Sequence[float], removed: Sequence[int],
                    t_w: float, phi: float, M: float, literal: bool = False) -> Tuple[float, List[int]]:
    """Eq. 3 for a given set of removed workers and wait time.  Returns (T_a,
    the removed workers whose gradients still arrive in time).  The test for
    "in time" has the form in which the candidate waits are built,
    child_time - t_ring <= t_w (the sum t_ring + t_w can round below
    child_time for t_w = child_time - t_ring)."""
    N = len(iter_time)
    ring = [w for w in range(N) if w not in removed]
    t_ring = max(iter_time[w] for w in ring)
    if literal:
        in_time = [w for w in removed if child_time[w] <= t_w]
    else:
        in_time = [w for w in removed if child_time[w] - t_ring <= t_w]
    x, q = len(removed), len(in_time)
    return (1.0 + phi / ((N - x + q) * M / N)) * (t_ring + t_w), in_time


def choose_all_reduce_mode(iter_time: Sequence[float], child_time: Sequence[float], phi: float, M: float,
                           t_w_max: float, threshold: float = 0.2):
    """Enumerate x = 0..X and the candidate waits; returns
    (x, t_w, T_a, removed workers, contributing workers sorted ascending)."""
    N = len(iter_time)
    slow_first = sorted(stragglers(iter_time, threshold), key=lambda w: (-iter_time[w], -w))
    best = None
    for x in range(0, min(len(slow_first), N - 1) + 1):
        removed = slow_first[:x]
        ring = [w for w in range(N) if w not in removed]
        t_ring = max(iter_time[w] for w in ring)
        waits = {0.0}
        for w in removed:
            need = child_time[w] - t_ring
            if 0.0 < need <= t_w_max:
                waits.add(need)
        for t_w in sorted(waits):
            T, in_time = time_all_reduce(iter_time, child_time, removed, t_w, phi, M)
            if best is None or T < best[2]:
                best = (x, t_w, T, list(removed), sorted(ring + in_time))
    return best
