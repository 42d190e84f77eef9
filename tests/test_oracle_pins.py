"""Pins for the CPU oracle: everything here checks ``oracle/`` against something
that is NOT the oracle — a hand-worked example, exact rational arithmetic,
closed forms of the recurrence, and PyTorch's library SGD optimizer."""
import itertools
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import star_oracle as O
from tests import exact_arith as X

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "worked_example.txt")


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns (round to nearest even), via torch."""
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def bf16_values(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32)


def csr(groups):
    off, mem = [0], []
    for g in groups:
        mem += list(g)
        off.append(len(mem))
    return np.array(off, np.int32), np.array(mem, np.int32)


def all_schedules(W):
    """Every ordered sequence of disjoint non-empty groups over subsets of the
    W workers, with every member order (partial covers included)."""
    for m in range(1, W + 1):
        for arrangement in itertools.permutations(range(W), m):
            for cuts in itertools.product([0, 1], repeat=m - 1):
                groups, cur = [], [arrangement[0]]
                for pos in range(1, m):
                    if cuts[pos - 1]:
                        groups.append(cur)
                        cur = []
                    cur.append(arrangement[pos])
                groups.append(cur)
                yield groups


# --------------------------------------------------------------------------
# 1. hand-worked example
# --------------------------------------------------------------------------
def _read_golden():
    scal, cases = {}, []
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line.startswith("case"):
            name, groups, p, v, trail = [s.strip() for s in line[4:].split("|")]
            groups = [[int(w) for w in g.split(",")] for g in groups.split(";")]
            cases.append((name, groups, float(p), float(v), [float(t) for t in trail.split()]))
        else:
            key, *vals = line.split()
            scal[key] = [float(x) for x in vals]
    return scal, cases


@pytest.mark.parametrize("variant", ["f32", "f64", "bf16"])
def test_hand_worked_example(variant):
    scal, cases = _read_golden()
    assert len(cases) == 4
    for name, groups, p_want, v_want, trail in cases:
        real = np.float64 if variant == "f64" else np.float32
        # 5 copies of the element: also checks that elements do not interact
        p = np.full(5, scal["p0"][0], real)
        v = np.full(5, scal["v0"][0], real)
        if variant == "bf16":     # 0.5, 0.25, -0.75, 1.5 are bf16-exact
            grads = [bf16_bits(np.full(5, g, np.float32)) for g in scal["g"]]
        else:
            grads = [np.full(5, g, np.float32) for g in scal["g"]]
        off, mem = csr(groups)
        snaps = [np.zeros(5, real) for _ in groups]
        fn = O.group_update_f64 if variant == "f64" else O.group_update_f32
        fn(p, v, grads, off, mem, scal["lr"][0], scal["mu"][0], scal["wd"][0], snapshots=snaps)
        assert np.all(p == p_want), name
        assert np.all(v == v_want), name
        for s, want in zip(snaps, trail):
            assert np.all(s == want), name


def test_summation_orders_on_the_hand_worked_example():
    scal, _ = _read_golden()
    g = [np.full(2, x, np.float32) for x in scal["order_g"]]
    for order, key in (("linear", "order_linear_p"), ("tree", "order_tree_p")):
        p, v = np.zeros(2, np.float32), np.zeros(2, np.float32)
        O.group_update_f32(p, v, g, [0, 4], [0, 1, 2, 3], 1.0, 0.0, 0.0, sum_order=order)
        assert np.all(p == np.float32(scal[key][0])), order
    assert scal["order_linear_p"][0] != scal["order_tree_p"][0]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_tree_order_brute_force_against_exact_pairwise_sums(dtype):
    """Every group size 1..9 (and 16, 17, 33), tree order, exact rounding."""
    rng = np.random.default_rng(21)
    n = 4
    for size in list(range(1, 10)) + [16, 17, 33]:
        W = size + 1
        p0 = rng.normal(0, 0.05, n).astype(np.float32)
        v0 = rng.normal(0, 0.02, n).astype(np.float32)
        g32 = [(rng.normal(0, 0.01, n) * 10.0 ** rng.integers(-3, 3)).astype(np.float32) for _ in range(W)]
        grads = [bf16_bits(g) for g in g32] if dtype == "bf16" else g32
        gval = [bf16_values(b) for b in grads] if dtype == "bf16" else g32
        members = [int(w) for w in rng.permutation(W)[:size]]
        groups = [members] if size < 3 else [members[:size - 1], members[size - 1:]]
        off, mem = csr(groups)
        p, v = p0.copy(), v0.copy()
        O.group_update_f32(p, v, grads, off, mem, np.float32(0.1), np.float32(0.9), np.float32(1e-4),
                           sum_order="tree")
        for i in range(n):
            pe, ve, _ = X.grouped_update_exact32(
                X.to_fraction(p0[i]), X.to_fraction(v0[i]), [X.to_fraction(gv[i]) for gv in gval], groups,
                [X.to_fraction(np.float32(0.1))] * len(groups), X.to_fraction(np.float32(0.9)),
                X.to_fraction(np.float32(1e-4)), tree=True)
            assert X.to_fraction(p[i]) == pe and X.to_fraction(v[i]) == ve, (size, i)


def test_tree_and_linear_orders_agree_up_to_rounding_and_exactly_for_small_groups():
    p0, v0, grads = _random_case(31, 3000, 9, "f32")
    for size in (1, 2):                      # one or two members: the same operations
        off, mem = csr([list(range(size))])
        a, b = p0.copy(), p0.copy()
        O.group_update_f32(a, v0.copy(), grads, off, mem, 0.1, 0.9, 1e-4, sum_order="linear")
        O.group_update_f32(b, v0.copy(), grads, off, mem, 0.1, 0.9, 1e-4, sum_order="tree")
        assert np.array_equal(a, b)
    off, mem = csr([list(range(9))])
    P, V = p0.astype(np.float64), v0.astype(np.float64)
    O.group_update_f64(P, V, grads, off, mem, 0.1, 0.9, 1e-4, sum_order="tree")
    a, b = p0.copy(), p0.copy()
    O.group_update_f32(a, v0.copy(), grads, off, mem, 0.1, 0.9, 1e-4, sum_order="linear")
    O.group_update_f32(b, v0.copy(), grads, off, mem, 0.1, 0.9, 1e-4, sum_order="tree")
    assert not np.array_equal(a, b)
    for x in (a, b):
        assert np.max(np.abs(x - P)) <= 16 * 2.0 ** -24 * 0.2


def bf16_snapshot_probe_values():
    """fp32 values that exercise the narrowing: random, exact ties with even and
    odd upper halves, just above / below ties, overflow to infinity, subnormals,
    signed zeros (infinite parameters turn into NaN through wd * p and cannot be
    held still)."""
    rng = np.random.default_rng(17)
    vals = [rng.normal(0, 1, 4096).astype(np.float32),
            (rng.normal(0, 1, 512) * 10.0 ** rng.integers(-30, 30, 512)).astype(np.float32)]
    upper = rng.integers(0x0001, 0x7F7F, 2048).astype(np.uint32) << 16
    for low in (0x8000, 0x7FFF, 0x8001, 0x0001, 0xFFFF):
        vals.append((upper | low).view(np.float32))
        vals.append((upper | low | 0x80000000).view(np.float32))
    special = np.array([0x7F7FFFFF, 0x7F7F8000, 0x7F7F7FFF, 0x00000001, 0x00008000, 0x00018000, 0x00007FFF,
                        0x00000000, 0x80000000], np.uint32).view(np.float32)
    vals.append(special)
    return np.concatenate(vals)


def test_bf16_snapshots_round_to_nearest_even_like_torch():
    """With zero gradients and zero momentum the parameters do not move, so the
    bf16 snapshot is the narrowing of the input: compare with PyTorch's cast."""
    x = bf16_snapshot_probe_values()
    n = x.size
    p, v = x.copy(), np.zeros(n, np.float32)
    snap = np.zeros(n, np.uint16)
    O.group_update_f32(p, v, [np.zeros(n, np.float32)], [0, 1], [0], 0.1, 0.9, 0.0, snapshots=[snap])
    assert np.array_equal(p.view(np.uint32), x.view(np.uint32))
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(snap, want)
    nan = np.array([np.nan], np.float32)
    s1 = np.zeros(1, np.uint16)
    O.group_update_f32(nan.copy(), np.zeros(1, np.float32), [np.zeros(1, np.float32)], [0, 1], [0], 0.1, 0.9, 0.0,
                       snapshots=[s1])
    assert np.isnan(bf16_values(s1))[0]


# --------------------------------------------------------------------------
# 2. exact-rational brute force: every schedule over W<=4, tiny n
# --------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_brute_force_every_schedule_exact_rounding(dtype):
    rng = np.random.default_rng(11)
    W, n = 4, 6
    p0 = rng.normal(0, 0.05, n).astype(np.float32)
    v0 = rng.normal(0, 0.02, n).astype(np.float32)
    g32 = rng.normal(0, 0.01, (W, n)).astype(np.float32)
    # a few awkward values: cancellation, subnormal, signed zero, large
    p0[0], g32[0][0], g32[1][0] = np.float32(1e-3), np.float32(0.0102), np.float32(0.0098)
    g32[2][1] = np.float32(1e-41)
    g32[3][2] = np.float32(-0.0)
    g32[1][3] = np.float32(3.0e4)
    if dtype == "bf16":
        grads = [bf16_bits(g) for g in g32]
        gval = [bf16_values(b) for b in grads]
    else:
        grads = [g.copy() for g in g32]
        gval = grads
    lr, mu, wd = np.float32(0.1), np.float32(0.9), np.float32(1e-4)
    count = 0
    for groups in all_schedules(W):
        count += 1
        lrs = [np.float32(lr * (1 + 0.25 * k)) for k in range(len(groups))]
        p, v = p0.copy(), v0.copy()
        snaps = [np.zeros(n, np.float32) for _ in groups]
        off, mem = csr(groups)
        O.group_update_f32(p, v, grads, off, mem, lrs, mu, wd, snapshots=snaps)
        for i in range(n):
            pe, ve, trail = X.grouped_update_exact32(
                X.to_fraction(p0[i]), X.to_fraction(v0[i]),
                [X.to_fraction(gv[i]) for gv in gval], groups,
                [X.to_fraction(l) for l in lrs], X.to_fraction(mu), X.to_fraction(wd))
            assert X.to_fraction(p[i]) == pe, (groups, i)
            assert X.to_fraction(v[i]) == ve, (groups, i)
            for k, t in enumerate(trail):
                assert X.to_fraction(snaps[k][i]) == t, (groups, i, k)
    assert count == 316


def test_brute_force_n_up_to_64_against_real_arithmetic():
    """f64 shadow vs the never-rounded rational recurrence, n = 1..64."""
    rng = np.random.default_rng(5)
    W = 5
    for n in (1, 2, 3, 7, 8, 9, 31, 33, 64):
        groups = [[4, 1], [0], [3, 2]]
        p0 = rng.normal(0, 0.05, n).astype(np.float32)
        v0 = rng.normal(0, 0.02, n).astype(np.float32)
        g32 = [rng.normal(0, 0.01, n).astype(np.float32) for _ in range(W)]
        lr, mu, wd = 0.1, 0.9, 1e-4
        p, v = p0.astype(np.float64), v0.astype(np.float64)
        off, mem = csr(groups)
        O.group_update_f64(p, v, g32, off, mem, lr, mu, wd)
        for i in range(n):
            pe, ve = X.grouped_update_real(
                Fraction(float(p0[i])), Fraction(float(v0[i])),
                [Fraction(float(g[i])) for g in g32], groups,
                [Fraction(lr)] * 3, Fraction(mu), Fraction(wd))
            assert abs(p[i] - float(pe)) <= 1e-14 * (abs(float(pe)) + 0.01)
            assert abs(v[i] - float(ve)) <= 1e-14 * (abs(float(ve)) + 0.01)


# --------------------------------------------------------------------------
# 3. closed forms
# --------------------------------------------------------------------------
def test_single_worker_no_momentum_no_decay_is_correctly_rounded_p_minus_lr_g():
    rng = np.random.default_rng(0)
    n = 4096
    p0 = rng.normal(0, 0.05, n).astype(np.float32)
    g = rng.normal(0, 0.01, n).astype(np.float32)
    lr = np.float32(0.1)
    p, v = p0.copy(), np.zeros(n, np.float32)
    O.group_update_f32(p, v, [g], [0, 1], [0], lr, 0.0, 0.0)
    assert np.array_equal(v, g)
    for i in range(n):
        want = X.round_binary32(X.to_fraction(p0[i]) - X.to_fraction(lr) * X.to_fraction(g[i]))
        assert X.to_fraction(p[i]) == want


def test_ssgd_equals_one_update_with_the_mean():
    """W a power of two and gradients on a coarse dyadic grid: sum and mean are
    exact, so the update equals the single-worker update on the mean, for every
    member order, bit for bit."""
    rng = np.random.default_rng(1)
    n, W = 1000, 8
    p0 = rng.normal(0, 0.05, n).astype(np.float32)
    v0 = rng.normal(0, 0.01, n).astype(np.float32)
    grads = [(rng.integers(-64, 65, n) / 1024.0).astype(np.float32) for _ in range(W)]
    mean = (np.sum(np.stack(grads).astype(np.float64), axis=0) / W).astype(np.float32)
    assert np.array_equal(mean.astype(np.float64) * W, np.sum(np.stack(grads).astype(np.float64), 0))
    lr, mu, wd = 0.1, 0.9, 1e-4
    ref_p, ref_v = p0.copy(), v0.copy()
    O.group_update_f32(ref_p, ref_v, [mean], [0, 1], [0], lr, mu, wd)
    for order in ([0, 1, 2, 3, 4, 5, 6, 7], [7, 6, 5, 4, 3, 2, 1, 0], [3, 0, 6, 1, 7, 2, 5, 4]):
        p, v = p0.copy(), v0.copy()
        O.group_update_f32(p, v, grads, [0, W], order, lr, mu, wd)
        assert np.array_equal(p, ref_p) and np.array_equal(v, ref_v)


def test_no_momentum_no_decay_sums_the_group_means():
    """mu = wd = 0: p_K = p_0 - lr * sum_k mean_k(g), v_K = mean_{K-1}."""
    rng = np.random.default_rng(2)
    n, W = 512, 6
    groups = [[5, 0], [2], [1, 3, 4]]
    p0 = rng.normal(0, 0.05, n)
    grads = [rng.normal(0, 0.01, n).astype(np.float32) for _ in range(W)]
    g64 = [g.astype(np.float64) for g in grads]
    means = [sum(g64[w] for w in grp) / len(grp) for grp in groups]
    lr = 0.1
    p, v = p0.copy(), rng.normal(0, 1, n)
    off, mem = csr(groups)
    O.group_update_f64(p, v, grads, off, mem, lr, 0.0, 0.0)
    np.testing.assert_allclose(p, p0 - lr * sum(means), rtol=0, atol=1e-16)
    np.testing.assert_allclose(v, means[-1], rtol=1e-15, atol=0)
    # and the fp32 sequence stays within its a-priori rounding bound of that
    p32, v32 = p0.astype(np.float32), np.zeros(n, np.float32)
    want = p32.astype(np.float64) - float(np.float32(lr)) * sum(means)
    O.group_update_f32(p32, v32, grads, off, mem, lr, 0.0, 0.0)
    assert np.max(np.abs(p32 - want)) <= 8 * 2.0 ** -24 * np.max(np.abs(want))


def test_no_decay_momentum_closed_form():
    """wd = 0: v_K = mu^K v_0 + sum_k mu^(K-1-k) gbar_k ; p_K = p_0 - lr sum_j v_j."""
    rng = np.random.default_rng(3)
    n, W = 257, 7
    groups = [[0, 6], [3], [1, 2], [5, 4]]
    K = len(groups)
    p0, v0 = rng.normal(0, 0.05, n), rng.normal(0, 0.02, n)
    grads = [rng.normal(0, 0.01, n).astype(np.float32) for _ in range(W)]
    g64 = [g.astype(np.float64) for g in grads]
    gbar = [sum(g64[w] for w in grp) / len(grp) for grp in groups]
    lr, mu = 0.05, 0.9
    vs = []
    for j in range(1, K + 1):
        vs.append(mu ** j * v0 + sum(mu ** (j - 1 - k) * gbar[k] for k in range(j)))
    p, v = p0.copy(), v0.copy()
    off, mem = csr(groups)
    O.group_update_f64(p, v, grads, off, mem, lr, mu, 0.0)
    np.testing.assert_allclose(v, vs[-1], rtol=1e-14, atol=1e-18)
    np.testing.assert_allclose(p, p0 - lr * sum(vs), rtol=1e-14, atol=1e-18)


def test_constant_gradient_is_a_2x2_affine_recurrence():
    """With the same mean gradient gbar in every group the state obeys
    [p; v] <- A [p; v] + b gbar with A = [[1 - lr wd, -lr mu], [wd, mu]],
    b = [-lr; 1]; K rounds = A^K x + (sum_j A^j) b gbar."""
    lr, mu, wd = 0.1, 0.9, 0.01
    A = np.array([[1 - lr * wd, -lr * mu], [wd, mu]])
    b = np.array([-lr, 1.0])
    K, n = 6, 33
    rng = np.random.default_rng(4)
    p0, v0 = rng.normal(0, 0.05, n), rng.normal(0, 0.02, n)
    g = rng.normal(0, 0.01, n).astype(np.float32)
    grads = [g.copy() for _ in range(K)]           # K workers, all the same gradient
    AK = np.linalg.matrix_power(A, K)
    S = sum(np.linalg.matrix_power(A, j) for j in range(K))
    want = AK @ np.stack([p0, v0]) + np.outer(S @ b, g.astype(np.float64))
    p, v = p0.copy(), v0.copy()
    O.group_update_f64(p, v, grads, list(range(K + 1)), list(range(K)), lr, mu, wd)
    np.testing.assert_allclose(p, want[0], rtol=1e-13, atol=1e-17)
    np.testing.assert_allclose(v, want[1], rtol=1e-13, atol=1e-17)


# --------------------------------------------------------------------------
# 4. a library routine: PyTorch's SGD optimizer, stepped once per group
# --------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_matches_torch_sgd_stepped_once_per_group(dtype):
    rng = np.random.default_rng(6)
    n, W = 300, 8
    groups = [[0, 1, 2], [3, 4, 5], [6, 7]]
    p0, v_unused = rng.normal(0, 0.05, n), None
    g32 = [rng.normal(0, 0.01, n).astype(np.float32) for _ in range(W)]
    if dtype == "bf16":
        grads = [bf16_bits(g) for g in g32]
        gval = [bf16_values(b).astype(np.float64) for b in grads]
    else:
        grads, gval = g32, [g.astype(np.float64) for g in g32]
    lr, mu, wd = 0.1, 0.9, 1e-4
    param = torch.nn.Parameter(torch.from_numpy(p0.copy()))
    opt = torch.optim.SGD([param], lr=lr, momentum=mu, weight_decay=wd, dampening=0,
                          nesterov=False)
    for rounds in range(2):                          # momentum carries across rounds
        for grp in groups:
            param.grad = torch.from_numpy(sum(gval[w] for w in grp) / len(grp))
            opt.step()
    p, v = p0.copy(), np.zeros(n)
    off, mem = csr(groups)
    for rounds in range(2):
        O.group_update_f64(p, v, grads, off, mem, lr, mu, wd)
    np.testing.assert_allclose(p, param.detach().numpy(), rtol=1e-13, atol=1e-17)
    buf = opt.state[param]["momentum_buffer"].numpy()
    np.testing.assert_allclose(v, buf, rtol=1e-13, atol=1e-17)


# --------------------------------------------------------------------------
# 5. invariants that tie the two variants and the fusion together
# --------------------------------------------------------------------------
def _random_case(seed, n, W, dtype):
    rng = np.random.default_rng(seed)
    p0 = rng.normal(0, 0.05, n).astype(np.float32)
    v0 = rng.normal(0, 0.02, n).astype(np.float32)
    g32 = [rng.normal(0, 0.01, n).astype(np.float32) for _ in range(W)]
    grads = [bf16_bits(g) for g in g32] if dtype == "bf16" else g32
    return p0, v0, grads


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_fused_groups_equal_successive_single_group_calls(dtype):
    p0, v0, grads = _random_case(7, 1031, 8, dtype)
    groups = [[2, 5, 7], [0], [1, 3], [6, 4]]
    lrs = [0.1, 0.05, 0.2, 0.025]
    off, mem = csr(groups)
    p, v = p0.copy(), v0.copy()
    snaps = [np.zeros_like(p0) for _ in groups]
    O.group_update_f32(p, v, grads, off, mem, lrs, 0.9, 1e-4, snapshots=snaps)
    q, u = p0.copy(), v0.copy()
    for k, grp in enumerate(groups):
        o1, m1 = csr([grp])
        O.group_update_f32(q, u, grads, o1, m1, lrs[k], 0.9, 1e-4)
        assert np.array_equal(snaps[k], q)
    assert np.array_equal(p, q) and np.array_equal(v, u)


def test_f32_sequence_tracks_the_f64_shadow():
    p0, v0, grads = _random_case(8, 20000, 16, "bf16")
    groups = [[0, 1, 2, 3], [4, 5, 6, 7], [8, 9, 10, 11], [12, 13, 14, 15]]
    off, mem = csr(groups)
    p, v = p0.copy(), v0.copy()
    P, V = p0.astype(np.float64), v0.astype(np.float64)
    lr, mu, wd = np.float32(1e-3), np.float32(0.9), np.float32(0.01)
    for _ in range(5):
        O.group_update_f32(p, v, grads, off, mem, lr, mu, wd)
        O.group_update_f64(P, V, grads, off, mem, float(lr), float(mu), float(wd))
    for a, b in ((p, P), (v, V)):
        rms = np.sqrt(np.mean(b * b))
        assert np.max(np.abs(a - b) / (np.abs(b) + rms)) < 1e-5


def test_member_permutation_changes_only_rounding():
    p0, v0, grads = _random_case(9, 5000, 6, "f32")
    lr, mu, wd = 0.1, 0.9, 1e-4
    P, V = p0.astype(np.float64), v0.astype(np.float64)
    O.group_update_f64(P, V, grads, [0, 6], [0, 1, 2, 3, 4, 5], lr, mu, wd)
    results = []
    for order in ([0, 1, 2, 3, 4, 5], [5, 3, 1, 0, 2, 4]):
        p, v = p0.copy(), v0.copy()
        O.group_update_f32(p, v, grads, [0, 6], order, lr, mu, wd)
        results.append(p)
        # |sum error| <= 5 ulp of the largest partial sum; then 3 roundings
        bound = 8 * 2.0 ** -24 * (np.abs(V) + np.abs(P) + 0.06)
        assert np.all(np.abs(p - P) <= bound) and np.all(np.abs(v - V) <= bound)
    assert not np.array_equal(results[0], results[1])     # rounding does differ somewhere


def test_group_order_matters_and_partial_cover_ignores_absent_workers():
    p0, v0, grads = _random_case(10, 100, 4, "f32")
    a, b = p0.copy(), p0.copy()
    O.group_update_f32(a, v0.copy(), grads, [0, 1, 2], [0, 1], 0.1, 0.9, 1e-2)
    O.group_update_f32(b, v0.copy(), grads, [0, 1, 2], [1, 0], 0.1, 0.9, 1e-2)
    assert not np.array_equal(a, b)
    c = p0.copy()
    O.group_update_f32(c, v0.copy(), [grads[0], grads[1], None, None], [0, 1, 2], [0, 1],
                       0.1, 0.9, 1e-2)
    assert np.array_equal(a, c)


def test_empty_schedule_and_empty_tensor_are_no_ops():
    p0, v0, grads = _random_case(12, 10, 2, "f32")
    p, v = p0.copy(), v0.copy()
    O.group_update_f32(p, v, grads, [0], [], 0.1, 0.9, 0.0)
    assert np.array_equal(p, p0) and np.array_equal(v, v0)
    e = np.zeros(0, np.float32)
    O.group_update_f32(e, e.copy(), [e.copy(), e.copy()], [0, 2], [0, 1], 0.1, 0.9, 0.0)


@pytest.mark.parametrize("off,mem", [([0, 0], []), ([0, 2], [0, 0]), ([0, 1], [3]),
                                      ([0, 1, 2], [1, 1]), ([0, 1], [-1])])
def test_rejects_schedules_outside_the_definition(off, mem):
    p0, v0, grads = _random_case(13, 4, 2, "f32")
    p = p0.copy()
    with pytest.raises(ValueError):
        O.group_update_f32(p, v0.copy(), grads, off, mem, 0.1, 0.9, 0.0)
    assert np.array_equal(p, p0)


def test_nan_and_inf_propagate_by_ieee_rules():
    p = np.array([1.0, 1.0, 1.0], np.float32)
    v = np.zeros(3, np.float32)
    g = [np.array([np.nan, np.inf, 1.0], np.float32), np.array([1.0, -np.inf, 1.0], np.float32)]
    O.group_update_f32(p, v, g, [0, 2], [0, 1], 0.5, 0.0, 0.0)
    assert np.isnan(p[0]) and np.isnan(p[1]) and p[2] == 0.5


def test_lr_rescale_makes_the_result_schedule_independent():
    """Section IV-C1: with r_new = (y / N) r_SSGD per update and mu = wd = 0,
    every schedule that covers all N workers lands on p_0 - (r / N) sum_w g_w."""
    from oracle import schedule as S
    rng = np.random.default_rng(14)
    n, N, r = 200, 8, 0.4
    p0 = rng.normal(0, 0.05, n)
    grads = [rng.normal(0, 0.01, n).astype(np.float32) for _ in range(N)]
    want = p0 - (r / N) * sum(g.astype(np.float64) for g in grads)
    for x in (1, 2, 3, 4, 8):
        off, mem = S.static_x(None, N, x)
        lrs = S.scaled_lrs(off, len(off) - 1, N, r)
        p, v = p0.copy(), np.zeros(n)
        O.group_update_f64(p, v, grads, off, mem, lrs, 0.0, 0.0)
        np.testing.assert_allclose(p, want, rtol=0, atol=1e-16)
