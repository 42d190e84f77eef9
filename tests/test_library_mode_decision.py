"""The library's host-side mode decision against the Python oracle."""
import random

import pytest

from oracle import mode_decision as D
from oracle import schedule as S
from paper_2512_09685_b200 import binding as B


def test_clustering_matches_oracle():
    rng = random.Random(0)
    for trial in range(200):
        W = rng.randint(1, 14)
        t = [rng.choice([0.2, 0.25, 0.5, 1.0]) + rng.random() * rng.choice([0.0, 0.01, 0.2]) for _ in range(W)]
        if trial % 7 == 0:
            t = [rng.choice([0.2, 0.4, 0.8]) for _ in range(W)]           # exact ties
        for k in (0, 1, 2, 3, W):
            assert B.star_cluster_iteration_times(t, k, -1.0) == D.agglomerative_clusters(t, n_clusters=k or None)
        for thr in (0.0, 0.05, 0.3):
            assert B.star_cluster_iteration_times(t, 0, thr) == D.agglomerative_clusters(t, max_distance=thr)
            assert B.star_cluster_iteration_times(t, 2, thr) == \
                D.agglomerative_clusters(t, n_clusters=2, max_distance=thr)


def test_mode_times_and_choice_match_oracle():
    rng = random.Random(1)
    chosen = set()
    for _ in range(300):
        W = rng.randint(1, 16)
        t = [rng.uniform(0.1, 0.5) * rng.choice([1, 1, 1, 4]) for _ in range(W)]
        labels = D.agglomerative_clusters(t, max_distance=0.1)
        phi, M = rng.choice([0.0, 10.0, 500.0, 1e5]), rng.choice([128.0, 1024.0])
        T_static, T_dynamic = B.star_mode_times(t, labels, phi, M)
        for x in range(1, W + 1):
            assert T_static[x - 1] == pytest.approx(D.time_static_x(t, x, phi, M), rel=1e-14)
        assert T_dynamic == pytest.approx(D.time_dynamic(t, labels, phi, M), rel=1e-14)
        x, T, (off, mem) = B.star_choose_mode(t, labels, phi, M)
        want_x, want_T = D.choose_mode(t, labels, phi, M)
        assert x == want_x and T == pytest.approx(want_T, rel=1e-14)
        chosen.add(min(x, 2) if x < W else "ssgd")
        if x == 0:
            assert (off, mem) == tuple(S.dynamic_x(t, labels))
        else:
            order = sorted(range(W), key=lambda w: (t[w], w))
            assert (off, mem) == tuple(S.static_x(order, W, x, sort_members=True))
        assert B.star_schedule_validate(off, mem, len(off) - 1, W) == B.STAR_OK
    assert len(chosen) >= 3                                     # dynamic, low-order and SSGD all occur


def test_worked_example_through_the_library():
    t = [1.0, 1.0, 2.0, 4.0]
    labels = B.star_cluster_iteration_times(t, 3)
    assert labels == [0, 0, 1, 2]
    T_static, T_dynamic = B.star_mode_times(t, labels, 64.0, 128.0)
    assert T_static == pytest.approx([3.0, 2.0, 10 / 3, 6.0]) and T_dynamic == pytest.approx(4 / 3)
    x, T, (off, mem) = B.star_choose_mode(t, labels, 64.0, 128.0)
    assert x == 0 and (off, mem) == ([0, 2, 3, 4], [0, 1, 2, 3])
    x, T, sched = B.star_choose_mode(t, None, 64.0, 128.0)      # without clusters: best static mode
    assert x == 2 and T == pytest.approx(2.0) and sched == ([0, 2, 4], [0, 1, 2, 3])


def test_mode_decision_rejects_bad_input():
    for t in ([0.0, 1.0], [-1.0, 1.0], [float("nan"), 1.0], [float("inf"), 1.0]):
        with pytest.raises(B.StarError):
            B.star_cluster_iteration_times(t, 1)
        with pytest.raises(B.StarError):
            B.star_mode_times(t, None, 1.0, 64.0)
    with pytest.raises(B.StarError):
        B.star_mode_times([1.0, 2.0], None, -1.0, 64.0)
    with pytest.raises(B.StarError):
        B.star_mode_times([1.0, 2.0], None, 1.0, 0.0)
    with pytest.raises(B.StarError):
        B.star_mode_times([1.0, 2.0], [0, -1], 1.0, 64.0)
    with pytest.raises(B.StarError):
        B.star_choose_mode([], None, 1.0, 64.0)


def test_all_reduce_mode_matches_oracle():
    rng = random.Random(4)
    seen_x = set()
    for _ in range(400):
        W = rng.randint(1, 12)
        t = [rng.uniform(0.1, 0.3) * rng.choice([1, 1, 1, 2, 6]) for _ in range(W)]
        child = [ti * rng.uniform(0.3, 1.0) for ti in t]
        phi, M, t_w_max = rng.choice([0.0, 5.0, 200.0, 1e5]), 512.0, rng.choice([0.0, 0.05, 0.5])
        x, t_w, T, removed, (off, mem) = B.star_choose_all_reduce_mode(t, child, phi, M, t_w_max)
        wx, wt, wT, wremoved, wused = D.choose_all_reduce_mode(t, child, phi, M, t_w_max)
        assert (x, removed, mem) == (wx, wremoved, wused) and off == [0, len(wused)]
        assert t_w == pytest.approx(wt, abs=1e-15) and T == pytest.approx(wT, rel=1e-14)
        assert B.star_schedule_validate(off, mem, 1, W) == B.STAR_OK
        seen_x.add(x)
    assert {0, 1, 2} <= seen_x


def test_all_reduce_worked_example_through_the_library():
    x, t_w, T, removed, sched = B.star_choose_all_reduce_mode([1.0, 1.0, 2.0, 4.0], [9.0, 9.0, 1.5, 3.0],
                                                              64.0, 128.0, 1.0)
    assert (x, t_w, removed, sched) == (2, 0.0, [3, 2], ([0, 2], [0, 1])) and T == pytest.approx(2.0)
    # children that are quick once attached and a noisy gradient (large phi): waiting for them pays,
    # (1 + phi/128) * 1.2 < (1 + phi/64) * 1
    x, t_w, T, removed, sched = B.star_choose_all_reduce_mode([1.0, 1.0, 2.0, 4.0], [9.0, 9.0, 1.1, 1.2],
                                                              1e4, 128.0, 1.0)
    assert (x, removed, sched) == (2, [3, 2], ([0, 4], [0, 1, 2, 3]))
    assert t_w == pytest.approx(0.2) and T == pytest.approx((1 + 1e4 / 128) * 1.2)
    with pytest.raises(B.StarError):
        B.star_choose_all_reduce_mode([1.0, 2.0], [1.0], 1.0, 64.0, 0.1)
    with pytest.raises(B.StarError):
        B.star_choose_all_reduce_mode([1.0, 2.0], [1.0, -2.0], 1.0, 64.0, 0.1)


def test_rounding_sensitive_wait_through_the_library():
    t_ring, child = 2.8929907811485323, 7.687996268929637
    t, c = [t_ring, t_ring] + [100.0] * 8, [1.0, 1.0] + [child] * 8
    x, t_w, T, removed, (off, mem) = B.star_choose_all_reduce_mode(t, c, 1e9, 64.0, 10.0)
    wx, wt, wT, wremoved, wused = D.choose_all_reduce_mode(t, c, 1e9, 64.0, 10.0)
    assert (x, removed, mem) == (8, wremoved, list(range(10))) == (wx, wremoved, wused)
    assert t_w == wt == child - t_ring and T == pytest.approx(wT, rel=1e-15)


def test_parent_assignment_matches_the_round_oracle():
    from oracle import all_reduce as AR
    rng = random.Random(8)
    for _ in range(200):
        W = rng.randint(1, 16)
        x = rng.randint(0, W - 1)
        removed = rng.sample(range(W), x)
        ring = [w for w in range(W) if w not in removed]
        want = AR.assign_parents(removed, ring)
        got = B.star_assign_parents(removed, W)
        assert got == [want.get(w, -1) for w in range(W)]
        counts = [got.count(r) for r in ring]
        assert max(counts) - min(counts) <= 1                      # children per parent balanced (Section IV-D2a)
    for removed, W in (([0, 0], 3), ([3], 3), ([0, 1, 2], 3)):
        with pytest.raises(B.StarError):
            B.star_assign_parents(removed, W)


def test_tree_construction_matches_the_round_oracle():
    from oracle import tree_round as TR
    rng = random.Random(9)
    for _ in range(300):
        W, fanout = rng.randint(0, 20), rng.randint(1, 5)
        latency = [float(rng.randint(0, 6)) for _ in range(W)]        # many ties
        assert B.star_build_tree(latency, fanout) == TR.build_tree(latency, fanout)
    with pytest.raises(B.StarError):
        B.star_build_tree([1.0, 2.0], 0)
    with pytest.raises(B.StarError):
        B.star_build_tree([1.0, float("nan")], 2)
