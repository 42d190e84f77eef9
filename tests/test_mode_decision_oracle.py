"""Pins for the mode-decision oracle: a hand-worked example of Eq. 1 / Eq. 2,
identities between the two equations, and SciPy's hierarchical clustering."""
import os

import numpy as np
import pytest
from scipy.cluster.hierarchy import fcluster, linkage

from oracle import mode_decision as D

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "mode_decision_example.txt")


def read_golden():
    out = {}
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        key, *vals = line.split()
        out[key] = [float(v) for v in vals]
    return out


def test_hand_worked_example():
    g = read_golden()
    t, M, phi = g["t"], g["M"][0], g["phi"][0]
    labels = [int(c) for c in g["clusters"]]
    for x, want in enumerate(g["T_static"], start=1):
        assert D.time_static_x(t, x, phi, M) == pytest.approx(want, rel=1e-14)
    assert D.time_dynamic(t, labels, phi, M) == pytest.approx(g["T_dynamic"][0], rel=1e-14)
    x, T = D.choose_mode(t, labels, phi, M)
    assert x == int(g["best_x"][0]) and T == pytest.approx(4 / 3, rel=1e-14)
    assert D.agglomerative_clusters(t, n_clusters=3) == labels


def test_eq2_with_one_cluster_is_eq1_at_x_equal_n():
    t = [0.3, 0.5, 0.25, 0.9, 0.4]
    assert D.time_dynamic(t, [0] * 5, 10.0, 640.0) == pytest.approx(D.time_static_x(t, 5, 10.0, 640.0))
    # SSGD: (1 + phi / M) * slowest worker
    assert D.time_static_x(t, 5, 10.0, 640.0) == pytest.approx((1 + 10 / 640) * 0.9)


def test_equal_workers_closed_form():
    """No stragglers, all N workers take t: T_x = (1 + phi N / (x M)) t falls with
    x, so SSGD is chosen (Section IV-B: a higher order has the lower TTA)."""
    N, t, M = 8, 0.2, 1024.0
    for phi in (1.0, 1e5):
        for x in range(1, N + 1):
            assert D.time_static_x([t] * N, x, phi, M) == pytest.approx((1 + phi * N / (x * M)) * t)
        assert D.choose_mode([t] * N, [0] * N, phi, M)[0] == N


def test_order_statistics_define_t_x():
    t = [0.7, 0.2, 0.9, 0.4]
    for x, want in zip((1, 2, 3, 4), (0.2, 0.4, 0.7, 0.9)):
        assert D.time_static_x(t, x, 0.0, 64.0) == pytest.approx(want)       # phi = 0: T_x = t_x


def test_a_straggler_pushes_the_choice_away_from_ssgd():
    t = [0.2] * 7 + [2.0]                      # one worker ten times slower
    labels = D.agglomerative_clusters(t, max_distance=0.1)
    assert labels == [0] * 7 + [1]
    x, T = D.choose_mode(t, labels, 2000.0, 1024.0)
    assert x == 0                              # dynamic: the seven fast workers synchronize among themselves
    assert T < D.time_static_x(t, 7, 2000.0, 1024.0) < D.time_static_x(t, 8, 2000.0, 1024.0)


def canonical(labels):
    seen, out = {}, []
    for l in labels:
        seen.setdefault(l, len(seen))
        out.append(seen[l])
    return out


@pytest.mark.parametrize("seed", range(20))
def test_clustering_matches_scipy_average_linkage(seed):
    rng = np.random.default_rng(seed)
    N = int(rng.integers(2, 17))
    t = rng.uniform(0.1, 1.0, N) + rng.choice([0.0, 1.0, 3.0], N)       # clumpy
    Z = linkage(t.reshape(-1, 1), method="average", metric="euclidean")
    for k in range(1, N + 1):
        want = canonical(fcluster(Z, k, criterion="maxclust"))
        got = D.agglomerative_clusters(list(t), n_clusters=k)
        assert got == want, (k, list(t))
    for thr in (0.05, 0.3, 1.5):
        want = canonical(fcluster(Z, thr, criterion="distance"))
        assert D.agglomerative_clusters(list(t), max_distance=thr) == want


# --------------------------------------------------------------------------
# all-reduce architecture, Eq. 3
# --------------------------------------------------------------------------
def test_straggler_rule_of_section_ii():
    assert D.deviation_ratios([1.0, 1.2, 1.21, 2.0]) == pytest.approx([0.0, 0.2, 0.21, 1.0])
    assert D.stragglers([1.0, 1.2, 1.21, 2.0]) == [2, 3]          # strictly more than 20 %


def test_all_reduce_hand_worked_example():
    g = read_golden()
    t, M, phi = g["t"], g["M"][0], g["phi"][0]
    child, t_w_max = g["ar_child_time"], g["ar_t_w_max"][0]
    assert D.time_all_reduce(t, child, [], 0.0, phi, M)[0] == pytest.approx(6.0)
    assert D.time_all_reduce(t, child, [3], 0.0, phi, M) == (pytest.approx(10 / 3), [])
    assert D.time_all_reduce(t, child, [3], 1.0, phi, M) == (pytest.approx(4.5), [3])
    assert D.time_all_reduce(t, child, [3, 2], 0.5, phi, M) == (pytest.approx(2.5), [2])
    x, t_w, T, removed, used = D.choose_all_reduce_mode(t, child, phi, M, t_w_max)
    assert (x, t_w, removed, used) == (int(g["ar_best_x"][0]), g["ar_best_t_w"][0], [3, 2], [0, 1])
    assert T == pytest.approx(g["ar_best_T"][0])


def test_eq3_without_removal_is_ssgd_eq1():
    t = [0.3, 0.5, 0.25, 0.9]
    T, used = D.time_all_reduce(t, t, [], 0.0, 12.0, 256.0)
    assert T == pytest.approx(D.time_static_x(t, 4, 12.0, 256.0)) and used == []


def test_breakpoint_enumeration_equals_a_dense_scan_of_wait_times():
    rng = np.random.default_rng(3)
    for _ in range(100):
        N = int(rng.integers(2, 9))
        t = list(rng.uniform(0.1, 0.3, N) * rng.choice([1, 1, 2, 5], N))
        child = [ti * rng.uniform(0.3, 1.0) for ti in t]
        phi, M, t_w_max = float(rng.choice([1.0, 50.0, 5000.0])), 512.0, 0.2
        x, t_w, T, removed, used = D.choose_all_reduce_mode(t, child, phi, M, t_w_max)
        slow = sorted(D.stragglers(t), key=lambda w: (-t[w], -w))
        dense = min(D.time_all_reduce(t, child, slow[:xx], tw, phi, M)[0]
                    for xx in range(0, min(len(slow), N - 1) + 1) for tw in np.linspace(0, t_w_max, 401))
        assert T <= dense * (1 + 1e-12)
        assert T == pytest.approx(D.time_all_reduce(t, child, removed, t_w, phi, M)[0])
        assert sorted(set(range(N)) - set(removed)) == [w for w in used if w not in removed]


def test_a_child_admitted_by_its_own_wait_exact_rational():
    """Eq. 3 over the rationals on an input where the float sum t_ring + t_w
    falls below the child's time for t_w = child_time - t_ring: the wait that is
    created for a child must admit that child (q = 1), as it does in exact
    arithmetic, and T_a must be the value Eq. 3 gives for N - x + q = N."""
    from fractions import Fraction
    t_ring, child = 2.8929907811485323, 7.687996268929637
    assert t_ring + (child - t_ring) < child                       # the rounding that used to drop the child
    # (by Sterbenz's lemma that needs child > 2 t_ring; waiting that long pays when many reports ride on it)
    N, x_want = 10, 8
    t = [t_ring, t_ring] + [100.0] * x_want                        # workers 2..9 are the stragglers
    child_time = [1.0, 1.0] + [child] * x_want
    phi, M = 1e9, 64.0                                             # noisy gradients: the eight reports are worth the wait
    x, t_w, T, removed, used = D.choose_all_reduce_mode(t, child_time, phi, M, t_w_max=10.0)
    assert (x, sorted(removed), used) == (x_want, list(range(2, N)), list(range(N)))
    assert t_w == child - t_ring
    F = Fraction
    exact = (1 + F(phi) / (F(N - x_want + x_want) * F(M) / N)) * (F(t_ring) + F(t_w))
    assert T == pytest.approx(float(exact), rel=1e-15)
    dropped = (1 + F(phi) / (F(N - x_want) * F(M) / N)) * (F(t_ring) + F(t_w))
    assert float(dropped) > T * 4                                  # what undercounting q would have reported


def test_where_the_literal_reading_of_q_parts_from_the_one_taken():
    """Read literally, a removed worker counts only if its whole iteration as a
    child fits into the wait t_w; the reading taken counts it if it is done t_w
    after the ring.  A child that needs 1.2 when the ring needs 1.0: a wait of
    0.2 admits it under the reading taken, not under the literal one (which
    would need a wait of 1.2, longer than a ring iteration)."""
    t, child, phi, M = [1.0, 1.0, 4.0], [9.0, 9.0, 1.2], 1e4, 128.0
    T_taken, in_taken = D.time_all_reduce(t, child, [2], 0.2, phi, M)
    T_literal, in_literal = D.time_all_reduce(t, child, [2], 0.2, phi, M, literal=True)
    assert in_taken == [2] and in_literal == []
    assert T_taken == pytest.approx((1 + phi / (3 * M / 3)) * 1.2)
    assert T_literal == pytest.approx((1 + phi / (2 * M / 3)) * 1.2)
    assert D.time_all_reduce(t, child, [2], 1.2, phi, M, literal=True)[1] == [2]
