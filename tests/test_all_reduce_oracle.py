"""Pins for the oracle of the all-reduce architecture (``oracle/all_reduce.py``,
``oracle_group_reduce_f32`` and ``oracle_update_from_sums_f32``): a hand-worked
example, exact rational arithmetic with explicit binary32 rounding over every
removal / lateness pattern of four workers, the special case that reduces to
the (separately pinned) SSGD update, real arithmetic, PyTorch's bf16 cast, and
planted mistakes that the pins must reject."""
import ctypes
import itertools
import os
import subprocess
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import all_reduce as AR
from oracle import star_oracle as O
from tests import exact_arith as X
from tests.test_oracle_pins import bf16_bits, bf16_snapshot_probe_values, bf16_values

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "all_reduce_example.txt")
SRC = os.path.join(os.path.dirname(O.__file__), "star_oracle.c")


def read_golden():
    removed, cases = [], []
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line.startswith("removed"):
            removed = [int(x) for x in line.split()[1:]]
        elif line.startswith("case"):
            name, g, late, scal, v, p = [s.strip() for s in line[4:].split("|")]
            cases.append((name, [float(x) for x in g.split()], [] if late == "-" else [int(x) for x in late.split()],
                          [float(x) for x in scal.split()], float(v), float(p)))
    return removed, cases


def exact_round(p, v, g, ring, parent_of, in_time, lr, mu, wd):
    """One element of the round over the rationals with one binary32 rounding
    per operation, written from the description, not from the oracle."""
    ring = sorted(ring)
    total = None
    for r in ring:
        a = g[r]
        for c in sorted(c for c in in_time if parent_of[c] == r):
            a = X.add32(a, g[c])
        total = a if total is None else X.add32(total, a)
    gbar = X.div32(total, Fraction(len(ring) + len(in_time)))
    d = X.fma32(wd, p, gbar)
    v = X.fma32(mu, v, d)
    p = X.fma32(-lr, v, p)
    return p, v


def patterns(W):
    """(removed in removal order, children in time) for every choice over W workers
    that leaves at least one ring member."""
    for x in range(0, W):
        for removed in itertools.permutations(range(W), x):
            for mask in itertools.product([0, 1], repeat=x):
                yield list(removed), [c for c, m in zip(removed, mask) if m]


# --------------------------------------------------------------------------
# the pins as one predicate over (round function), so that mutants can be fed in
# --------------------------------------------------------------------------
def pins_accept(round_fn, reduce_fn=O.group_reduce_f32, stride=1) -> bool:
    removed, cases = read_golden()
    for as_bf16 in (False, True):
        for name, g, late, (p0, v0, lr, mu, wd), v_want, p_want in cases:
            ring = [w for w in range(len(g)) if w not in removed]
            parent_of = AR.assign_parents(removed, ring)
            grads = [np.full(3, x, np.float32) for x in g]
            if as_bf16:
                grads = [bf16_bits(x) for x in grads]
            p, v = np.full(3, p0, np.float32), np.full(3, v0, np.float32)
            round_fn(p, v, grads, ring, parent_of, [c for c in removed if c not in late], lr, mu, wd)
            if not (np.all(p == np.float32(p_want)) and np.all(v == np.float32(v_want))):
                return False
    # exact-rational brute force, four workers, awkward values in the mix
    rng = np.random.default_rng(11)
    W, n = 4, 6
    p0 = rng.normal(0, 0.05, n).astype(np.float32)
    v0 = rng.normal(0, 0.02, n).astype(np.float32)
    g32 = [rng.normal(0, 0.01, n).astype(np.float32) for _ in range(W)]
    g32[0][0], g32[1][0], g32[2][0], g32[3][0] = 1.0, 2.0 ** -24, 2.0 ** -24, -1.0      # cancellation and ties
    g32[0][1], g32[1][1], g32[2][1], g32[3][1] = 1e-41, -0.0, 3e38, 1e-45               # subnormals, large
    bits = [bf16_bits(g) for g in g32]
    lr, mu, wd = np.float32(0.1), np.float32(0.9), np.float32(1e-3)
    for grads, vals in ((g32, g32), (bits, [bf16_values(b) for b in bits])):
        for index, (removed, in_time) in enumerate(patterns(W)):
            if index % stride:
                continue
            ring = [w for w in range(W) if w not in removed]
            parent_of = AR.assign_parents(removed, ring)
            p, v = p0.copy(), v0.copy()
            round_fn(p, v, grads, ring, parent_of, in_time, lr, mu, wd)
            for i in range(n):
                pe, ve = exact_round(X.to_fraction(p0[i]), X.to_fraction(v0[i]), [X.to_fraction(g[i]) for g in vals],
                                     ring, parent_of, in_time, X.to_fraction(lr), X.to_fraction(mu),
                                     X.to_fraction(wd))
                if X.to_fraction(p[i]) != pe or X.to_fraction(v[i]) != ve:
                    return False
    # the parent's aggregate alone: listed order, pairwise order, bf16 output
    for size in (1, 2, 3, 5, 7):
        gs = [rng.normal(0, 0.01, n).astype(np.float32) for _ in range(size + 1)]
        members = list(rng.permutation(size + 1)[:size])
        lin = reduce_fn(gs, members)
        tree = reduce_fn(gs, members, sum_order="tree")
        for i in range(n):
            want = X.to_fraction(gs[members[0]][i])
            for m in members[1:]:
                want = X.add32(want, X.to_fraction(gs[m][i]))
            if X.to_fraction(lin[i]) != want:
                return False
            if X.to_fraction(tree[i]) != X.pairwise_sum32([X.to_fraction(gs[m][i]) for m in members]):
                return False
    x = bf16_snapshot_probe_values()
    if not np.array_equal(reduce_fn([x], [0], out_dtype="bf16"),
                          torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)):
        return False
    return True


def test_hand_worked_example_and_brute_force():
    assert pins_accept(AR.all_reduce_round_f32)


def test_golden_values_are_what_the_file_says():
    removed, cases = read_golden()
    assert removed == [4, 3] and [c[0] for c in cases] == ["all_in_time", "one_late", "order"]
    # the "order" case: the plain worker-order sum loses both small terms
    g = [np.float32(x) for x in cases[2][1]]
    plain = ((g[0] + g[1]) + g[2]) + g[4]
    assert plain == np.float32(1.5)
    assert np.float32(cases[2][4]) * 4 == np.float32(1.5) + np.float32(2.0 ** -23)


# --------------------------------------------------------------------------
# special cases that reduce to something pinned elsewhere
# --------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_nobody_removed_is_the_ssgd_update(dtype):
    """Ring = all workers in index order, no children: aggregate r is worker r's
    gradient, the ring sum is the left-to-right sum, the divisor is N: bit for
    bit the one-group update of oracle_group_update_f32."""
    rng = np.random.default_rng(5)
    n, W = 257, 6
    p0 = rng.normal(0, 0.05, n).astype(np.float32)
    v0 = rng.normal(0, 0.02, n).astype(np.float32)
    grads = [rng.normal(0, 0.01, n).astype(np.float32) for _ in range(W)]
    if dtype == "bf16":
        grads = [bf16_bits(g) for g in grads]
    p, v = p0.copy(), v0.copy()
    aggregates, n_reports = AR.all_reduce_round_f32(p, v, grads, range(W), {}, [], 0.1, 0.9, 1e-3)
    assert n_reports == W and len(aggregates) == W
    q, u = p0.copy(), v0.copy()
    O.group_update_f32(q, u, grads, [0, W], list(range(W)), np.float32(0.1), 0.9, 1e-3)
    assert np.array_equal(p.view(np.uint32), q.view(np.uint32))
    assert np.array_equal(v.view(np.uint32), u.view(np.uint32))


def test_exact_sums_make_the_round_a_group_update_over_the_contributors():
    """Gradients on a coarse dyadic grid add without rounding in any order, so
    the round equals one group update over ring + children in time, whatever
    the parent assignment; late children change nothing."""
    rng = np.random.default_rng(6)
    n, W = 100, 7
    grads = [(rng.integers(-64, 65, n) / 256.0).astype(np.float32) for _ in range(W)]
    p0 = rng.normal(0, 0.05, n).astype(np.float32)
    v0 = rng.normal(0, 0.02, n).astype(np.float32)
    removed, in_time = [6, 2, 4], [2, 6]
    ring = [0, 1, 3, 5]
    want_p, want_v = p0.copy(), v0.copy()
    contributors = sorted(ring + in_time)
    O.group_update_f32(want_p, want_v, grads, [0, len(contributors)], contributors, np.float32(0.05), 0.9, 1e-2)
    for parent_of in (AR.assign_parents(removed, ring), {6: 5, 2: 5, 4: 5}, {6: 0, 2: 3, 4: 1}):
        p, v = p0.copy(), v0.copy()
        poisoned = list(grads)
        poisoned[4] = np.full(n, np.nan, np.float32)          # the late child's gradient is never read
        _, n_reports = AR.all_reduce_round_f32(p, v, poisoned, ring, parent_of, in_time, 0.05, 0.9, 1e-2)
        assert n_reports == 6
        assert np.array_equal(p.view(np.uint32), want_p.view(np.uint32))
        assert np.array_equal(v.view(np.uint32), want_v.view(np.uint32))


def test_round_tracks_real_arithmetic():
    rng = np.random.default_rng(7)
    n, W = 64, 8
    p0 = rng.normal(0, 0.05, n).astype(np.float32)
    v0 = rng.normal(0, 0.02, n).astype(np.float32)
    grads = [rng.normal(0, 0.01, n).astype(np.float32) for _ in range(W)]
    removed, in_time = [7, 5, 1], [7, 1]
    ring = [0, 2, 3, 4, 6]
    p, v = p0.copy(), v0.copy()
    AR.all_reduce_round_f32(p, v, grads, ring, AR.assign_parents(removed, ring), in_time, 0.1, 0.9, 1e-3)
    lr, mu, wd = (X.to_fraction(np.float32(x)) for x in (0.1, 0.9, 1e-3))
    for i in range(n):
        pe, ve = X.grouped_update_real(X.to_fraction(p0[i]), X.to_fraction(v0[i]),
                                       [X.to_fraction(g[i]) for g in grads], [sorted(ring + in_time)], [lr], mu, wd)
        assert abs(float(pe) - float(p[i])) <= 1e-6 * (abs(float(pe)) + 0.05)
        assert abs(float(ve) - float(v[i])) <= 1e-6 * (abs(float(ve)) + 0.02)


def test_parents_are_dealt_round_robin_over_the_ring():
    assert AR.assign_parents([], [0, 1]) == {}
    assert AR.assign_parents([7, 5, 6], [2, 0]) == {7: 0, 5: 2, 6: 0}
    assert AR.assign_parents([3], [2, 1, 0]) == {3: 0}
    kids = AR.children_of({7: 0, 5: 2, 6: 0}, [6, 7])
    assert kids == {0: [6, 7]}


def test_one_member_aggregate_is_the_exact_widening():
    bits = np.arange(0, 65536, 7, dtype=np.uint16)
    out = O.group_reduce_f32([None, bits], [1])
    assert np.array_equal(out.view(np.uint32), bits.astype(np.uint32) << 16)


def test_arguments_outside_the_definition_are_rejected():
    g = [np.zeros(4, np.float32), np.zeros(4, np.float32)]
    for members in ([], [0, 0], [2], [-1]):
        with pytest.raises(ValueError):
            O.group_reduce_f32(g, members)
    p, v = np.zeros(4, np.float32), np.zeros(4, np.float32)
    with pytest.raises(ValueError):
        O.update_from_sums_f32(p, v, [], 1, 0.1, 0.9, 0.0)
    with pytest.raises(ValueError):
        O.update_from_sums_f32(p, v, [g[0], g[1]], 1, 0.1, 0.9, 0.0)      # fewer reports than partial sums


# --------------------------------------------------------------------------
# planted mistakes (in copies, on the CPU): the pins above must notice each
# --------------------------------------------------------------------------
C_MUTANTS = {
    "divides_by_ring_size": ("const float gbar = s / (float)n_reports;", "const float gbar = s / (float)R;"),
    "reciprocal_multiply": ("const float gbar = s / (float)n_reports;",
                            "const float gbar = s * (1.0f / (float)n_reports);"),
    "ring_sum_right_to_left": ("float s = sums[0][i];\n        for (int r = 1; r < R; ++r)\n            s = s + sums[r][i];",
                               "float s = sums[R - 1][i];\n        for (int r = R - 2; r >= 0; --r)\n            s = s + sums[r][i];"),
    "last_ring_member_dropped": ("for (int r = 1; r < R; ++r)", "for (int r = 1; r < R - 1; ++r)"),
    "weight_decay_dropped": ("const float d = fmaf(wd, params[i], gbar);", "const float d = gbar;"),
    "momentum_not_fused": ("const float v = fmaf(mu, momentum[i], d);", "const float v = mu * momentum[i] + d;"),
    "ascent": ("params[i] = fmaf(-lr, v, params[i]);", "params[i] = fmaf(lr, v, params[i]);"),
    "step_before_momentum_store": ("params[i] = fmaf(-lr, v, params[i]);", "params[i] = fmaf(-lr, d, params[i]);"),
    "aggregate_skips_last_child": ("for (int j = 1; j < count; ++j)\n                s = s + grad_at(grads[members[j]], grad_dtype, i);",
                                   "for (int j = 1; j < count - 1; ++j)\n                s = s + grad_at(grads[members[j]], grad_dtype, i);"),
    "aggregate_indexes_by_position": ("s = s + grad_at(grads[members[j]], grad_dtype, i);\n        }\n        if (out_dtype",
                                      "s = s + grad_at(grads[j], grad_dtype, i);\n        }\n        if (out_dtype"),
    "aggregate_bf16_truncates": ("u += 0x7fffu + ((u >> 16) & 1u);", "u += 0u;"),
}

PY_MUTANTS = {
    "children_before_parent": ("[r] + kids.get(r, [])", "kids.get(r, []) + [r]"),
    "late_children_counted": ("n_reports = len(ring) + len(in_time)", "n_reports = len(ring) + len(parent_of)"),
    "late_children_summed": ("for c in sorted(in_time):", "for c in sorted(parent_of):"),
    "ring_in_given_order": ("ring = sorted(int(r) for r in ring)", "ring = [int(r) for r in ring][::-1]"),
    "children_descending": ("for c in sorted(in_time):", "for c in sorted(in_time, reverse=True):"),
}


def c_mutant(tmp_path, name):
    text = open(SRC).read()
    old, new = C_MUTANTS[name]
    assert text.count(old) >= 1, "mutation site not found: " + name
    # mutate the LAST occurrence: the all-reduce functions are at the end of the file
    head, _, tail = text.rpartition(old)
    if name == "aggregate_bf16_truncates":
        head, _, tail = text.partition(old)
    path = tmp_path / (name + ".c")
    path.write_text(head + new + tail)
    lib_path = str(tmp_path / (name + ".so"))
    subprocess.check_call(["gcc", *[f for f in O.CFLAGS if f not in ("-Wall", "-Wextra")], "-o", lib_path,
                           str(path), "-lm"])
    lib = ctypes.CDLL(lib_path)
    lib.oracle_group_reduce_f32.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_int, ctypes.c_int,
                                            ctypes.c_int64, ctypes.c_void_p, ctypes.c_int, ctypes.c_int]
    lib.oracle_update_from_sums_f32.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int,
                                                ctypes.c_int64, ctypes.c_int, ctypes.c_float, ctypes.c_float,
                                                ctypes.c_float]
    return lib


class _Swapped:
    """star_oracle's front end with the C library replaced by a mutant build."""

    def __init__(self, lib):
        self.lib = lib

    def __enter__(self):
        self.saved = O._lib
        O._load()
        self.saved = O._lib
        O._lib = self.lib
        return self

    def __exit__(self, *exc):
        O._lib = self.saved


def test_pins_reject_c_mutants(tmp_path):
    for name in sorted(C_MUTANTS):
        lib = c_mutant(tmp_path, name)
        with _Swapped(lib):
            assert not pins_accept(AR.all_reduce_round_f32, stride=3), "the pins did not notice: " + name
    assert pins_accept(AR.all_reduce_round_f32, stride=3)


def test_pins_reject_composition_mutants():
    text = open(AR.__file__).read()
    for name, (old, new) in sorted(PY_MUTANTS.items()):
        assert text.count(old) == 1, "mutation site not found: " + name
        scope = {"__name__": "oracle.all_reduce_mutant", "__package__": "oracle"}
        exec(compile(text.replace(old, new), name, "exec"), scope)
        assert not pins_accept(scope["all_reduce_round_f32"], stride=3), "the pins did not notice: " + name
