"""GPU parity on small tensors: every tail length, misaligned bases, every
schedule over four workers, wide schedules, non-finite values, error paths."""
import itertools

import numpy as np
import pytest
import torch

from oracle import star_oracle as O
from tests.parity import assert_matches, grad_to_numpy

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2512_09685_b200 import binding
    return binding


def make_case(n, W, dtype, seed, offset=0, pad=64):
    """Buffers carved out of larger NaN-filled allocations at `offset` elements,
    so that out-of-range writes are seen and misaligned bases are exercised."""
    g = torch.Generator(device="cuda").manual_seed(seed)
    def carve(dt, std):
        raw = torch.full((n + 2 * pad + offset,), float("nan"), dtype=dt, device="cuda")
        view = raw[pad + offset: pad + offset + n]
        view.copy_(torch.randn(n, generator=g, device="cuda") * std)
        return raw, view
    p_raw, p = carve(torch.float32, 0.05)
    v_raw, v = carve(torch.float32, 0.02)
    grads = [carve(dtype, 0.01) for _ in range(W)]
    return (p_raw, p), (v_raw, v), grads


def run_both(B, p, v, grads, off, mem, lr, mu, wd):
    p_np, v_np = p.cpu().numpy().copy(), v.cpu().numpy().copy()
    g_np = [None if g is None else grad_to_numpy(g) for g in grads]
    O.group_update_f32(p_np, v_np, g_np, off, mem, np.float32(lr), mu, wd)
    B.star_group_update(p, v, grads, off, mem, lr, mu, wd)
    torch.cuda.synchronize()
    return p_np, v_np


def guards_intact(raw, view_len, offset, pad=64):
    head = raw[: pad + offset]
    tail = raw[pad + offset + view_len:]
    return bool(torch.isnan(head.float()).all()) and bool(torch.isnan(tail.float()).all())


SIZES = list(range(1, 70)) + [127, 128, 129, 255, 256, 257, 4095, 4096, 4097, 8191, 8193,
                              65535, 65537, 1_000_003]


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_every_tail_length(B, dtype):
    off, mem = [0, 3, 4, 6], [4, 0, 2, 5, 1, 3]
    for n in SIZES:
        (p_raw, p), (v_raw, v), grads = make_case(n, 6, dtype, seed=n)
        want_p, want_v = run_both(B, p, v, [g for _, g in grads], off, mem, 0.1, 0.9, 1e-4)
        assert_matches(p, want_p, "p n=%d" % n)
        assert_matches(v, want_v, "v n=%d" % n)
        assert guards_intact(p_raw, n, 0) and guards_intact(v_raw, n, 0)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_misaligned_bases_take_the_scalar_path_with_identical_results(B, dtype):
    off, mem = [0, 2, 3], [1, 0, 2]
    for offset in range(0, 17):
        for n in (1, 13, 300, 5000):
            (p_raw, p), (v_raw, v), grads = make_case(n, 3, dtype, seed=offset * 100 + n, offset=offset)
            want_p, want_v = run_both(B, p, v, [g for _, g in grads], off, mem, 0.1, 0.9, 1e-4)
            assert_matches(p, want_p, "p off=%d n=%d" % (offset, n))
            assert_matches(v, want_v, "v off=%d n=%d" % (offset, n))
            assert guards_intact(p_raw, n, offset) and guards_intact(v_raw, n, offset)
            for raw, g in grads:                       # gradients are never written
                assert guards_intact(raw, n, offset)


def test_only_one_buffer_misaligned(B):
    n = 4099
    (_, p), (_, v), grads = make_case(n, 2, torch.bfloat16, seed=5)
    shifted = torch.empty(n + 1, dtype=torch.bfloat16, device="cuda")[1:]
    shifted.copy_(grads[1][1])
    want_p, want_v = run_both(B, p, v, [grads[0][1], shifted], [0, 2], [0, 1], 0.1, 0.9, 1e-4)
    assert_matches(p, want_p, "p")
    assert_matches(v, want_v, "v")


def all_schedules(W):
    for m in range(1, W + 1):
        for arrangement in itertools.permutations(range(W), m):
            for cuts in itertools.product([0, 1], repeat=m - 1):
                off, mem = [0], []
                for pos, w in enumerate(arrangement):
                    if pos > 0 and cuts[pos - 1]:
                        off.append(len(mem))
                    mem.append(w)
                off.append(len(mem))
                yield off, mem


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_every_schedule_over_four_workers(B, dtype):
    n = 61
    (_, p0), (_, v0), grads = make_case(n, 4, dtype, seed=77)
    gl = [g for _, g in grads]
    count = 0
    for off, mem in all_schedules(4):
        p, v = p0.clone(), v0.clone()
        want_p, want_v = run_both(B, p, v, gl, off, mem, 0.1, 0.9, 1e-4)
        assert_matches(p, want_p, "p %r %r" % (off, mem))
        assert_matches(v, want_v, "v %r %r" % (off, mem))
        count += 1
    assert count == 316


@pytest.mark.parametrize("W", [1, 7, 8, 9, 16, 17, 32, 33, 63, 64])
def test_wide_random_schedules(B, W):
    rng = np.random.default_rng(W)
    n = 10_007
    (_, p0), (_, v0), grads = make_case(n, W, torch.bfloat16, seed=W)
    gl = [g for _, g in grads]
    for trial in range(6):
        m = int(rng.integers(1, W + 1)) if trial else W
        mem = [int(w) for w in rng.permutation(W)[:m]]
        cuts = sorted(set(int(c) for c in rng.integers(1, m, size=int(rng.integers(0, m)))) ) if m > 1 else []
        off = [0] + cuts + [m]
        if trial == 1:
            off = list(range(m + 1))                    # ASGD
        if trial == 2:
            off = [0, m]                                # SSGD
        used = [g if w in mem else None for w, g in enumerate(gl)]
        p, v = p0.clone(), v0.clone()
        want_p, want_v = run_both(B, p, v, used, off, mem, 0.05, 0.9, 5e-4)
        assert_matches(p, want_p, "p W=%d trial=%d" % (W, trial))
        assert_matches(v, want_v, "v W=%d trial=%d" % (W, trial))


def test_fused_call_equals_one_call_per_group(B):
    n = 33_333
    (_, p0), (_, v0), grads = make_case(n, 8, torch.bfloat16, seed=3)
    gl = [g for _, g in grads]
    groups = [[0, 1, 2], [3, 4, 5], [6, 7]]
    off, mem = [0, 3, 6, 8], [0, 1, 2, 3, 4, 5, 6, 7]
    p, v = p0.clone(), v0.clone()
    B.star_group_update(p, v, gl, off, mem, 0.1, 0.9, 1e-4)
    q, u = p0.clone(), v0.clone()
    for grp in groups:
        B.star_group_update(q, u, gl, [0, len(grp)], grp, 0.1, 0.9, 1e-4)
    torch.cuda.synchronize()
    assert torch.equal(p, q) and torch.equal(v, u)


def test_closed_form_single_worker(B):
    """One worker, mu = wd = 0: p' is the correctly rounded p - lr g (a single
    fused multiply-add), v' = g."""
    n = 100_000
    (_, p), (_, v), grads = make_case(n, 1, torch.float32, seed=9)
    g = grads[0][1]
    want = torch.addcmul(p.double(), g.double(), torch.tensor(-float(np.float32(0.1)),
                         dtype=torch.float64, device="cuda")).float()      # exact product, one rounding
    B.star_group_update(p, v, [g], [0, 1], [0], 0.1, 0.0, 0.0)
    torch.cuda.synchronize()
    assert torch.equal(v, g)
    # double rounding (53 -> 24 bits) can differ from the fused result in rare ties only
    assert (p != want).float().mean().item() < 1e-6


def test_non_finite_values_and_signed_zero(B):
    n = 64
    p = torch.ones(n, device="cuda")
    v = torch.zeros(n, device="cuda")
    g0 = torch.zeros(n, device="cuda")
    g1 = torch.zeros(n, device="cuda")
    g0[0], g1[0] = float("nan"), 1.0
    g0[1], g1[1] = float("inf"), float("-inf")
    g0[2], g1[2] = float("inf"), 1.0
    g0[3], g1[3] = -0.0, -0.0
    g0[4], g1[4] = 1e-41, 1e-41                        # subnormal
    g0[5], g1[5] = 3e38, 3e38                          # the sum overflows
    p[3] = 0.0
    want_p, want_v = run_both(B, p, v, [g0, g1], [0, 2], [0, 1], 0.5, 0.0, 0.0)
    assert_matches(p, want_p, "p")
    assert_matches(v, want_v, "v")
    got_v = v.cpu().numpy()
    assert np.signbit(got_v[3]) == np.signbit(want_v[3])
    p2, v2 = torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda")
    gneg = torch.full((n,), -0.0, device="cuda")
    want_p, want_v = run_both(B, p2, v2, [gneg], [0, 1], [0], 0.5, 0.0, 0.0)
    assert np.array_equal(np.signbit(v2.cpu().numpy()), np.signbit(want_v))
    assert np.array_equal(np.signbit(p2.cpu().numpy()), np.signbit(want_p))


def test_errors_leave_state_untouched(B):
    n = 1000
    (_, p), (_, v), grads = make_case(n, 4, torch.bfloat16, seed=21)
    gl = [g for _, g in grads]
    p0, v0 = p.clone(), v.clone()
    bad = [([0, 0, 2], [0, 1]), ([0, 2], [1, 1]), ([0, 1], [4]), ([1, 2], [0, 1]), ([0, 1], [-1])]
    for off, mem in bad:
        with pytest.raises(B.StarError) as e:
            B.star_group_update(p, v, gl, off, mem, 0.1, 0.9, 0.0)
        assert e.value.status == B.STAR_ERR_BAD_SCHEDULE
    with pytest.raises(B.StarError) as e:
        B.star_group_update(p, v, [gl[0], None, None, None], [0, 2], [0, 1], 0.1, 0.9, 0.0)
    assert e.value.status == B.STAR_ERR_NULL_POINTER
    with pytest.raises(B.StarError) as e:                      # params and momentum overlap
        B.star_group_update(p, p[: n], gl, [0, 1], [0], 0.1, 0.9, 0.0)
    assert e.value.status == B.STAR_ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert torch.equal(p, p0) and torch.equal(v, v0)
    # no-ops
    B.star_group_update(p, v, gl, [0], [], 0.1, 0.9, 0.0)
    e0 = torch.empty(0, device="cuda")
    B.star_group_update(e0, e0.clone(), [torch.empty(0, device="cuda")], [0, 1], [0], 0.1, 0.9, 0.0)
    torch.cuda.synchronize()
    assert torch.equal(p, p0) and torch.equal(v, v0)


def test_runs_on_a_side_stream_and_counts_launches(B):
    n = 50_000
    (_, p), (_, v), grads = make_case(n, 2, torch.bfloat16, seed=31)
    gl = [g for _, g in grads]
    p_np, v_np = p.cpu().numpy().copy(), v.cpu().numpy().copy()
    before = B.star_launch_count()
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        for _ in range(3):
            B.star_group_update(p, v, gl, [0, 1, 2], [1, 0], 0.1, 0.9, 1e-4)
    s.synchronize()
    assert B.star_launch_count() - before == 3
    g_np = [grad_to_numpy(g) for g in gl]
    for _ in range(3):
        O.group_update_f32(p_np, v_np, g_np, [0, 1, 2], [1, 0], np.float32(0.1), 0.9, 1e-4)
    assert_matches(p, p_np, "p")
    assert_matches(v, v_np, "v")


def test_rounds_captured_in_a_cuda_graph_replay_correctly(B):
    """The flat entry point only enqueues one kernel on the given stream, so a
    sequence of rounds can be captured once and replayed (launch-bound small
    tensors).  Three rounds with different schedules, replayed twice."""
    n = 65_537
    (_, p), (_, v), grads = make_case(n, 4, torch.bfloat16, seed=41)
    gl = [g for _, g in grads]
    schedules = [([0, 2, 4], [0, 1, 2, 3]), ([0, 1, 2, 3, 4], [3, 1, 0, 2]), ([0, 4], [2, 3, 0, 1])]
    p_np, v_np = p.cpu().numpy().copy(), v.cpu().numpy().copy()
    g_np = [grad_to_numpy(g) for g in gl]
    B.star_group_update(p, v, gl, *schedules[0], 0.1, 0.9, 1e-4)          # warm-up outside the capture
    O.group_update_f32(p_np, v_np, g_np, *schedules[0], np.float32(0.1), 0.9, 1e-4)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            for off, mem in schedules:
                B.star_group_update(p, v, gl, off, mem, 0.1, 0.9, 1e-4)
    # capturing does not execute: state is still the warm-up result
    assert_matches(p, p_np, "p after capture")
    for _ in range(2):
        graph.replay()
        for off, mem in schedules:
            O.group_update_f32(p_np, v_np, g_np, off, mem, np.float32(0.1), 0.9, 1e-4)
    torch.cuda.synchronize()
    assert_matches(p, p_np, "p after replays")
    assert_matches(v, v_np, "v after replays")


def test_concurrent_host_threads_on_their_own_streams(B):
    """The library keeps per-device launch geometry in shared caches; two host
    threads issuing rounds on their own streams and tensors must not disturb
    each other."""
    import threading
    n, rounds = 40_003, 25
    cases = []
    for t in range(2):
        (_, p), (_, v), grads = make_case(n, 3, torch.bfloat16 if t == 0 else torch.float32, seed=50 + t)
        cases.append((p, v, [g for _, g in grads], ([0, 1, 3], [2, 0, 1]) if t == 0 else ([0, 3], [1, 2, 0])))
    expected = []
    for p, v, gl, (off, mem) in cases:
        p_np, v_np = p.cpu().numpy().copy(), v.cpu().numpy().copy()
        g_np = [grad_to_numpy(g) for g in gl]
        for _ in range(rounds):
            O.group_update_f32(p_np, v_np, g_np, off, mem, np.float32(0.05), 0.9, 1e-4)
        expected.append((p_np, v_np))
    torch.cuda.synchronize()
    errors = []

    def worker(idx):
        try:
            p, v, gl, (off, mem) = cases[idx]
            stream = torch.cuda.Stream()
            with torch.cuda.stream(stream):
                for _ in range(rounds):
                    B.star_group_update(p, v, gl, off, mem, 0.05, 0.9, 1e-4)
            stream.synchronize()
        except Exception as exc:                       # surfaced below
            errors.append(exc)

    threads = [threading.Thread(target=worker, args=(i,)) for i in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    for (p, v, _, _), (p_np, v_np) in zip(cases, expected):
        assert_matches(p, p_np, "params")
        assert_matches(v, v_np, "momentum")


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_sparse_gradients_with_exact_and_signed_zeros(B, dtype):
    """Group sums that are exactly +0 or -0 (unused rows, dead units) take a
    shortcut around the division in the kernel: the mean must still be the
    IEEE quotient, sign of zero included."""
    n, W = 50_001, 6
    (_, p), (_, v), grads = make_case(n, W, dtype, seed=61)
    gl = [g for _, g in grads]
    g = torch.Generator(device="cuda").manual_seed(62)
    keep = torch.rand(n, generator=g, device="cuda") < 0.3          # 70 % of the elements: all workers zero
    negz = torch.rand(n, generator=g, device="cuda") < 0.5
    for x in gl:
        x.mul_(keep.to(x.dtype))
        x.copy_(torch.where(~keep & negz, torch.full_like(x, -0.0), x))
    gl[2][::7] = 0.0                                                 # mixed signs of zero inside a group
    p[::11] = 0.0
    off, mem = [0, 3, 4, 6], [0, 1, 2, 3, 4, 5]
    for wd in (0.0, 1e-4):
        q, u = p.clone(), v.clone().zero_()
        want_p, want_v = run_both(B, q, u, gl, off, mem, 0.1, 0.0 if wd == 0.0 else 0.9, wd)
        assert_matches(q, want_p, "p wd=%g" % wd)
        assert_matches(u, want_v, "v wd=%g" % wd)
        assert np.array_equal(np.signbit(u.cpu().numpy()), np.signbit(want_v))
        assert np.array_equal(np.signbit(q.cpu().numpy()), np.signbit(want_p))


def test_buffers_marshalled_once_give_the_same_rounds(B):
    """FlatRoundBuffers forwards to the same entry point with the same pointers."""
    n = 70_001
    (_, p), (_, v), grads = make_case(n, 5, torch.bfloat16, seed=31)
    gl = [g for _, g in grads]
    q, u = p.clone(), v.clone()
    rounds = B.FlatRoundBuffers(q, u, gl)
    for off, mem in (([0, 2, 5], [4, 1, 0, 2, 3]), ([0, 1, 2], [3, 0]), ([0, 5], [0, 1, 2, 3, 4])):
        B.star_group_update(p, v, gl, off, mem, 0.1, 0.9, 1e-4)
        rounds.star_group_update(off, mem, 0.1, 0.9, 1e-4)
    torch.cuda.synchronize()
    assert torch.equal(p, q) and torch.equal(v, u)


@pytest.mark.parametrize("size", [2, 3, 4, 5, 8, 16, 32, 64])
def test_group_means_on_extreme_sums(B, size):
    """The mean of a group whose sum is subnormal, on a rounding tie of the
    quotient, huge, infinite, NaN or a signed zero: power-of-two group sizes take a
    multiply by 2^-k in the kernel, the others the IEEE division; both must land
    on the oracle's s / |G| bit for bit (mu = wd = 0, lr = 1: v = mean, p = p0 - mean)."""
    probes = np.array([0.0, -0.0, 1e-45, -1e-45, 3e-45, 5e-45, 7e-45, 1.1754944e-38, 1.1754942e-38, 2.3509887e-38,
                       -2.9387359e-38, 1.0, 1.0 + 2.0 ** -23, 3.0, -7.0, 1e-20, 3.4028235e38, -3.4028235e38,
                       np.inf, -np.inf, np.nan, 8.5e37, 2.0 ** -126 * 1.5, 2.0 ** -127, 2.0 ** -149 * (size + 1)],
                      np.float32)
    n = probes.size
    # the first member carries the probe, the others are zero: the group's sum IS the probe
    grads = [torch.from_numpy(probes.copy()).cuda()] + [torch.zeros(n, device="cuda") for _ in range(size - 1)]
    off, mem = [0, size], list(range(size))
    for sum_order, name in ((B.STAR_SUM_LINEAR, "linear"), (B.STAR_SUM_TREE, "tree")):
        p, v = torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda")
        p_np, v_np = np.zeros(n, np.float32), np.zeros(n, np.float32)
        O.group_update_f32(p_np, v_np, [g.cpu().numpy() for g in grads], off, mem, np.float32(1.0), 0.0, 0.0,
                           sum_order=name)
        B.star_group_update_ex(p, v, grads, off, mem, [1.0], 0.0, 0.0, sum_order=sum_order)
        torch.cuda.synchronize()
        got_v, got_p = v.cpu().numpy(), p.cpu().numpy()
        nan = np.isnan(v_np)
        assert np.array_equal(np.isnan(got_v), nan) and np.array_equal(np.isnan(got_p), np.isnan(p_np))
        assert np.array_equal(got_v[~nan].view(np.uint32), v_np[~nan].view(np.uint32)), (size, name)
        ok = ~np.isnan(p_np)
        assert np.array_equal(got_p[ok].view(np.uint32), p_np[ok].view(np.uint32)), (size, name)
        want = probes.astype(np.float64) / size                    # and the oracle's mean is the rounded quotient
        finite = np.isfinite(want) & ~nan
        assert np.array_equal(v_np[finite], want[finite].astype(np.float32))
