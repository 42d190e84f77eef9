"""Pins for the schedule oracle: mode definitions of Sections I, IV-B, IV-C1."""
import itertools

import pytest

from oracle import schedule as S


def groups_of(sched):
    off, mem = sched
    return [mem[off[k]:off[k + 1]] for k in range(len(off) - 1)]


def test_ssgd_is_one_group_of_all_and_asgd_is_singletons_in_arrival_order():
    assert groups_of(S.static_x(None, 8, 8)) == [[0, 1, 2, 3, 4, 5, 6, 7]]
    order = [3, 1, 7, 0, 2, 6, 5, 4]
    assert groups_of(S.static_x(order, 8, 1)) == [[w] for w in order]


@pytest.mark.parametrize("x", [1, 2, 4, 8])
def test_x_order_modes_of_the_eight_worker_experiment(x):
    """Section IV-B runs 1-, 2-, 4- and 8-order modes on N = 8 workers: each
    update uses x gradients, so a round has 8 / x updates."""
    g = groups_of(S.static_x(None, 8, x))
    assert len(g) == 8 // x and all(len(grp) == x for grp in g)
    assert sorted(itertools.chain(*g)) == list(range(8))


def test_static_x_ragged_tail_and_member_sorting():
    order = [5, 2, 7, 0, 1, 6, 3, 4]
    assert groups_of(S.static_x(order, 8, 3)) == [[5, 2, 7], [0, 1, 6], [3, 4]]
    assert groups_of(S.static_x(order, 8, 3, sort_members=True)) == [[2, 5, 7], [0, 1, 6], [3, 4]]
    # partial cover: only five workers arrived
    assert groups_of(S.static_x([4, 0, 3, 9, 1], 10, 2)) == [[4, 0], [3, 9], [1]]


def test_from_labels_orders_groups_by_label_and_skips_absent_workers():
    assert groups_of(S.from_labels([0, 0, 0, 1, 1, 1, 2, 2])) == [[0, 1, 2], [3, 4, 5], [6, 7]]
    assert groups_of(S.from_labels([2, -1, 0, 2, 0, 7])) == [[2, 4], [0, 3], [5]]
    assert S.from_labels([-1, -1]) == ([0], [])


def test_dynamic_x_sorts_clusters_by_their_slowest_member():
    # cluster 0 = {0, 3} (slowest 0.9), cluster 1 = {1, 2} (slowest 0.4), cluster 2 = {4} (0.5)
    t = [0.2, 0.4, 0.3, 0.9, 0.5]
    c = [0, 1, 1, 0, 2]
    assert groups_of(S.dynamic_x(t, c)) == [[1, 2], [4], [0, 3]]
    # a tie in the maximum: the cluster holding the smaller worker index first
    assert groups_of(S.dynamic_x([0.5, 0.5, 0.1], [1, 0, 1])) == [[0, 2], [1]]
    # brute force: every output is sorted by max time and is a valid schedule
    for labels in itertools.product([0, 1, 2, -1], repeat=4):
        times = [0.3, 0.1, 0.4, 0.15]
        off, mem = S.dynamic_x(times, labels)
        K = len(off) - 1
        assert S.is_valid(off, mem, K, 4)
        maxes = [max(times[w] for w in grp) for grp in groups_of((off, mem))]
        assert maxes == sorted(maxes)
        assert sorted(mem) == [w for w, l in enumerate(labels) if l >= 0]


def test_is_valid():
    assert S.is_valid([0, 2, 4], [0, 1, 2, 3], 2, 4)
    assert S.is_valid([0], [], 0, 4)
    assert S.is_valid([0, 1], [2], 1, 4)                 # partial cover
    assert not S.is_valid([0, 0, 2], [0, 1], 2, 4)       # empty group
    assert not S.is_valid([0, 2], [1, 1], 1, 4)          # duplicate
    assert not S.is_valid([0, 1, 2], [1, 1], 2, 4)       # duplicate across groups
    assert not S.is_valid([0, 1], [4], 1, 4)             # out of range
    assert not S.is_valid([1, 2], [0, 1], 1, 4)          # offsets must start at 0
    assert not S.is_valid([0, 2, 1], [0, 1], 2, 4)       # offsets must increase


def test_scaled_lrs_follow_reports_per_update():
    off, _ = S.static_x(None, 8, 3)
    assert S.scaled_lrs(off, 3, 8, 0.8) == pytest.approx([0.3, 0.3, 0.2])
