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
