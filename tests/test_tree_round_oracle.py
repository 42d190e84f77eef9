"""Pins for the oracle of a round over a communication tree
(``oracle/tree_round.py``): hand-worked examples, exact rational arithmetic
with explicit binary32 rounding over every rooted forest on four workers, the
special cases that reduce to separately pinned routines (a flat tree is the
SSGD update in worker order; a chain is a right-to-left sum), real arithmetic,
the layer-by-layer construction against its definition, and planted mistakes
that the pins must reject."""
import itertools
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import star_oracle as O
from oracle import tree_round as TR
from tests import exact_arith as X
from tests.test_oracle_pins import bf16_bits, bf16_values

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "tree_round_example.txt")


def read_golden():
    cases = []
    for line in open(GOLDEN):
        line = line.strip()
        if not line.startswith("case"):
            continue
        name, lat, fan, parents, g, scal, v, p = [s.strip() for s in line[4:].split("|")]
        cases.append((name, [float(x) for x in lat.split()], int(fan), [int(x) for x in parents.split()],
                      [float(x) for x in g.split()], [float(x) for x in scal.split()], float(v), float(p)))
    return cases


def forests(W):
    """Every parent array over W workers in which each worker reaches the root (-1)."""
    for parents in itertools.product(range(-1, W), repeat=W):
        ok = True
        for w in range(W):
            seen, node = 0, w
            while node != -1 and seen <= W:
                node, seen = parents[node], seen + 1
            ok = ok and node == -1
        if ok and all(parents[w] != w for w in range(W)):
            yield list(parents)


def exact_round(p, v, g, parent_of, lr, mu, wd):
    """One element of the round over the rationals with one binary32 rounding
    per operation, written from the description, not from the oracle."""
    W = len(parent_of)

    def forwarded(w):
        s = g[w]
        for c in range(W):                      # ascending worker index
            if parent_of[c] == w:
                s = X.add32(s, forwarded(c))
        return s
    total = None
    for w in range(W):
        if parent_of[w] == -1:
            total = forwarded(w) if total is None else X.add32(total, forwarded(w))
    gbar = X.div32(total, Fraction(W))
    d = X.fma32(wd, p, gbar)
    v = X.fma32(mu, v, d)
    p = X.fma32(-lr, v, p)
    return p, v


def pins_accept(round_fn, build_fn=TR.build_tree, stride=1) -> bool:
    for as_bf16 in (False, True):
        for name, lat, fan, parents, g, (p0, v0, lr, mu, wd), v_want, p_want in read_golden():
            if build_fn(lat, fan) != parents:
                return False
            grads = [np.full(3, x, np.float32) for x in g]
            if as_bf16:
                grads = [bf16_bits(x) for x in grads]
            p, v = np.full(3, p0, np.float32), np.full(3, v0, np.float32)
            round_fn(p, v, grads, parents, lr, mu, wd)
            if not (np.all(p == np.float32(p_want)) and np.all(v == np.float32(v_want))):
                return False
    rng = np.random.default_rng(17)
    W, n = 4, 6
    p0 = rng.normal(0, 0.05, n).astype(np.float32)
    v0 = rng.normal(0, 0.02, n).astype(np.float32)
    g32 = [rng.normal(0, 0.01, n).astype(np.float32) for _ in range(W)]
    g32[0][0], g32[1][0], g32[2][0], g32[3][0] = 1.0, 2.0 ** -24, 2.0 ** -24, -1.0      # cancellation and ties
    g32[0][1], g32[1][1], g32[2][1], g32[3][1] = 1e-41, -0.0, 3e38, 1e-45               # subnormals, large
    bits = [bf16_bits(g) for g in g32]
    lr, mu, wd = np.float32(0.1), np.float32(0.9), np.float32(1e-3)
    count = 0
    for grads, vals in ((g32, g32), (bits, [bf16_values(b) for b in bits])):
        for index, parents in enumerate(forests(W)):
            count += 1
            if index % stride:
                continue
            p, v = p0.copy(), v0.copy()
            round_fn(p, v, grads, parents, lr, mu, wd)
            for i in range(n):
                pe, ve = exact_round(X.to_fraction(p0[i]), X.to_fraction(v0[i]), [X.to_fraction(x[i]) for x in vals],
                                     parents, X.to_fraction(lr), X.to_fraction(mu), X.to_fraction(wd))
                if X.to_fraction(p[i]) != pe or X.to_fraction(v[i]) != ve:
                    return False
    assert count == 2 * 125                      # (W + 1)^(W - 1) rooted forests on 4 labelled workers
    return True


def test_hand_worked_examples_and_brute_force():
    assert pins_accept(TR.tree_round_f32)


def test_golden_values_are_what_the_file_says():
    cases = {c[0]: c for c in read_golden()}
    assert set(cases) == {"two_levels", "order", "chain"}
    assert cases["order"][6] == 0.375 + 2.0 ** -25 and cases["order"][7] == -(0.1875 + 2.0 ** -26)
    assert cases["order"][4][:2] == [2.0 ** -24, 2.0 ** -24]


@pytest.mark.parametrize("as_bf16", [False, True])
def test_a_flat_tree_is_the_ssgd_update_in_worker_order(as_bf16):
    """Every worker a child of the root: S = g_0 + g_1 + ... left to right, mean
    over N -- the single-group update of the (separately pinned) grouped oracle."""
    rng = np.random.default_rng(2)
    n, W = 257, 7
    grads = [rng.normal(0, 0.01, n).astype(np.float32) for _ in range(W)]
    if as_bf16:
        grads = [bf16_bits(g) for g in grads]
    p, v = rng.normal(0, 0.05, n).astype(np.float32), rng.normal(0, 0.02, n).astype(np.float32)
    q, u = p.copy(), v.copy()
    TR.tree_round_f32(p, v, grads, [-1] * W, 0.1, 0.9, 1e-3)
    O.group_update_f32(q, u, grads, [0, W], list(range(W)), np.float32(0.1), 0.9, 1e-3)
    assert np.array_equal(p.view(np.uint32), q.view(np.uint32)) and np.array_equal(v.view(np.uint32), u.view(np.uint32))


def test_a_chain_sums_from_the_far_end():
    """root <- 0 <- 1 <- 2 <- 3: s_0 = g_0 + (g_1 + (g_2 + g_3)), in exact arithmetic with binary32 rounding."""
    vals = [1.0, 2.0 ** -24, 2.0 ** -24, 2.0 ** -24]
    grads = [np.full(2, x, np.float32) for x in vals]
    sums = TR.partial_sums_f32(grads, [-1, 0, 1, 2])
    want = X.add32(Fraction(vals[0]), X.add32(Fraction(vals[1]), X.add32(Fraction(vals[2]), Fraction(vals[3]))))
    assert X.to_fraction(sums[0][0]) == want == Fraction(1) + Fraction(2) ** -22     # the small terms survive together
    left_to_right = Fraction(1)                                                       # ((1 + e) + e) + e loses them all
    for x in vals[1:]:
        left_to_right = X.add32(left_to_right, Fraction(x))
    assert left_to_right == 1


def test_round_tracks_real_arithmetic():
    rng = np.random.default_rng(4)
    n, W = 500, 9
    grads = [rng.normal(0, 0.01, n).astype(np.float32) for _ in range(W)]
    parents = TR.build_tree(list(rng.uniform(0, 1, W)), 2)
    p0, v0 = rng.normal(0, 0.05, n).astype(np.float32), rng.normal(0, 0.02, n).astype(np.float32)
    p, v = p0.copy(), v0.copy()
    TR.tree_round_f32(p, v, grads, parents, 0.1, 0.9, 1e-3)
    gbar = sum(g.astype(np.float64) for g in grads) / W
    v_real = 0.9 * v0.astype(np.float64) + (gbar + 1e-3 * p0.astype(np.float64))
    p_real = p0.astype(np.float64) - 0.1 * v_real
    assert np.max(np.abs(v - v_real)) <= 1e-6 * np.max(np.abs(v_real))
    assert np.max(np.abs(p - p_real)) <= 1e-6 * np.max(np.abs(p_real))


def test_tree_is_filled_layer_by_layer_in_ascending_latency():
    rng = np.random.default_rng(6)
    for _ in range(200):
        W, k = int(rng.integers(1, 20)), int(rng.integers(1, 5))
        lat = [float(x) for x in rng.integers(0, 6, W)]               # many ties
        parents = TR.build_tree(lat, k)
        order = sorted(range(W), key=lambda w: (lat[w], w))
        depth = {}
        for w in order:                                               # parents come earlier in the order
            depth[w] = 0 if parents[w] == -1 else depth[parents[w]] + 1
        kids = TR.children_lists(parents)
        assert len(kids[-1]) == min(k, W)                             # the k quickest hang off the root
        assert all(len(kids[w]) <= k for w in range(W))
        for w in range(W):
            if parents[w] != -1:                                      # nobody hangs below a slower worker
                assert (lat[parents[w]], parents[w]) < (lat[w], w)
        by_depth = [depth[w] for w in order]
        assert by_depth == sorted(by_depth)                           # slower workers are never higher up
        level_sizes = [by_depth.count(d) for d in range(max(by_depth) + 1)]
        assert all(level_sizes[d] == k ** (d + 1) for d in range(len(level_sizes) - 1))   # full layers above the last
    with pytest.raises(ValueError):
        TR.build_tree([1.0], 0)
    with pytest.raises(ValueError):
        TR.partial_sums_f32([np.zeros(1, np.float32)] * 2, [1, 0])   # a cycle


PY_MUTANTS = {
    "children_before_own": ("parts = [own] + [visit(c, depth + 1) for c in kids[w]]",
                            "parts = [visit(c, depth + 1) for c in kids[w]] + [own]"),
    "children_descending": ("out[int(p)].append(w)", "out[int(p)].insert(0, w)"),
    "mean_over_root_children": ("[sums[w] for w in top], len(parent_of), lr", "[sums[w] for w in top], len(top), lr"),
    "grandchildren_dropped": ("parts = [own] + [visit(c, depth + 1) for c in kids[w]]",
                              "parts = [own] + [O.group_reduce_f32([grads[c]], [0]) for c in kids[w]]"),
    "slowest_first": ("key=lambda w: (latency[w], w))", "key=lambda w: (-latency[w], w))"),
    "parent_is_previous_worker": ("parent_of[w] = order[(i - fanout) // fanout]", "parent_of[w] = order[i - fanout]"),
}


def test_pins_reject_composition_mutants():
    text = open(TR.__file__).read()
    for name, (old, new) in sorted(PY_MUTANTS.items()):
        assert text.count(old) >= 1, "mutation site not found: " + name
        scope = {"__name__": "oracle.tree_round_mutant", "__package__": "oracle"}
        exec(compile(text.replace(old, new), name, "exec"), scope)
        assert not pins_accept(scope["tree_round_f32"], scope["build_tree"], stride=2), \
            "the pins did not notice: " + name
