"""All-reduce architecture on the GPU (Section IV-B, Eq. 3): the parent's local
aggregate (``star_group_reduce``) and the update from the ring members'
aggregates (``star_group_update_from_sums``) against the CPU oracle, bit for
bit, and a whole round composed from them against ``oracle/all_reduce.py``."""
import numpy as np
import pytest
import torch

from oracle import all_reduce as AR
from oracle import star_oracle as O
from tests.parity import assert_matches, grad_to_numpy

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2512_09685_b200 import binding
    return binding


PAD = 64


def carve(n, dtype, offset, fill):
    """A view of n elements at `offset` elements into a NaN-padded allocation."""
    raw = torch.full((n + 2 * PAD + offset,), float("nan"), dtype=dtype, device="cuda")
    view = raw[PAD + offset: PAD + offset + n]
    view.copy_(fill)
    return raw, view


def guards_intact(raw, n, offset):
    return bool(torch.isnan(raw[: PAD + offset].float()).all()) and bool(
        torch.isnan(raw[PAD + offset + n:].float()).all())


def bits(t):
    return t.cpu().view(torch.int16).numpy().view(np.uint16)


def check_reduce(B, grads, members, out_dtype, order, n, out_offset=0, what=""):
    g_np = [grad_to_numpy(g) for g in grads]
    want = O.group_reduce_f32(g_np, members, out_dtype="bf16" if out_dtype == torch.bfloat16 else "f32",
                              sum_order="tree" if order else "linear")
    raw, out = carve(n, out_dtype, out_offset, torch.zeros(n, device="cuda"))
    before = B.star_launch_count()
    B.star_group_reduce(out, grads, members, sum_order=order)
    torch.cuda.synchronize()
    assert B.star_launch_count() == before + 1
    if out_dtype == torch.bfloat16:
        assert np.array_equal(bits(out), want), what
    else:
        assert_matches(out, want, what)
    assert guards_intact(raw, n, out_offset), what


SIZES = list(range(1, 20)) + [31, 32, 33, 255, 256, 257, 2047, 2048, 2049, 4099, 65537, 1_000_003]


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])
def test_reduce_every_tail_length(B, dtype, out_dtype):
    W = 6
    for n in SIZES:
        gen = torch.Generator(device="cuda").manual_seed(n)
        grads = [(torch.randn(n, generator=gen, device="cuda") * 0.01).to(dtype) for _ in range(W)]
        for order in (B.STAR_SUM_LINEAR, B.STAR_SUM_TREE):
            check_reduce(B, grads, [4, 0, 5, 2, 1], out_dtype, order, n, what="n=%d order=%d" % (n, order))
        check_reduce(B, grads, [3, 5], out_dtype, B.STAR_SUM_LINEAR, n, what="n=%d two members" % n)
        check_reduce(B, grads, [1], out_dtype, B.STAR_SUM_LINEAR, n, what="n=%d one member" % n)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_reduce_group_sizes_in_both_orders(B, dtype):
    """1..9, 16, 17, 33 and 64 members: every kernel variant of the tree order."""
    rng = np.random.default_rng(3)
    for count in list(range(1, 10)) + [15, 16, 17, 31, 33, 63, 64]:
        W = min(64, count + 3)
        for n in (7, 4099, 150_001):
            gen = torch.Generator(device="cuda").manual_seed(count * 13 + n)
            grads = [(torch.randn(n, generator=gen, device="cuda") * 0.01).to(dtype) for _ in range(W)]
            members = [int(w) for w in rng.permutation(W)[:count]]
            for order in (B.STAR_SUM_LINEAR, B.STAR_SUM_TREE):
                check_reduce(B, grads, members, torch.float32, order, n, what="count=%d n=%d" % (count, n))


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_reduce_at_every_alignment(B, dtype):
    """Sources and output at a common element offset (vector body after a short
    head) and at differing offsets (element path): same bits either way."""
    for n in (5, 300, 5003):
        for offset in range(0, 17):
            gen = torch.Generator(device="cuda").manual_seed(offset * 31 + n)
            fills = [torch.randn(n, generator=gen, device="cuda") * 0.01 for _ in range(4)]
            for spread in (0, 1):                                   # 0: congruent, 1: every buffer its own offset
                carved = [carve(n, dtype, offset + spread * w, f) for w, f in enumerate(fills)]
                grads = [view for _, view in carved]
                for out_dtype in (torch.float32, torch.bfloat16):
                    for members in ([2, 0, 3, 1], [3, 1], [2]):     # [3, 1] and [2]: the two-vectors-per-thread kernel
                        check_reduce(B, grads, members, out_dtype, B.STAR_SUM_LINEAR, n, out_offset=offset,
                                     what="n=%d offset=%d spread=%d members=%r" % (n, offset, spread, members))
                for w, (raw, _) in enumerate(carved):
                    assert guards_intact(raw, n, offset + spread * w)


def test_reduce_special_values(B):
    """Signed zeros, infinities, NaN and sums that round on the way."""
    vals = np.array([0.0, -0.0, 1.0, -1.0, np.inf, -np.inf, np.nan, 2.0 ** -24, 1.0 + 2.0 ** -23, 3e38, -3e38,
                     1e-45, -1e-45], np.float32)
    grid = np.array(np.meshgrid(vals, vals, vals)).reshape(3, -1)
    grads = [torch.from_numpy(grid[w].copy()).cuda() for w in range(3)]
    n = grid.shape[1]
    for members in ([0, 1, 2], [2, 0], [1]):
        want = O.group_reduce_f32([g.cpu().numpy() for g in grads], members)
        out = torch.empty(n, device="cuda")
        B.star_group_reduce(out, grads, members)
        torch.cuda.synchronize()
        got = out.cpu().numpy()
        assert np.array_equal(np.isnan(got), np.isnan(want))
        ok = ~np.isnan(want)
        assert np.array_equal(got[ok].view(np.uint32), want[ok].view(np.uint32))    # signed zeros included


def test_reduce_errors(B):
    n = 100
    grads = [torch.zeros(n, device="cuda") for _ in range(3)]
    out = torch.zeros(n, device="cuda")
    before = B.star_launch_count()
    for members, status in (([], B.STAR_ERR_BAD_SCHEDULE), ([0, 0], B.STAR_ERR_BAD_SCHEDULE),
                            ([3], B.STAR_ERR_BAD_SCHEDULE), ([-1], B.STAR_ERR_BAD_SCHEDULE)):
        with pytest.raises(B.StarError) as e:
            B.star_group_reduce(out, grads, members)
        assert e.value.status == status
    with pytest.raises(B.StarError) as e:                            # output overlaps a listed source
        B.star_group_reduce(grads[1], grads, [0, 1])
    assert e.value.status == B.STAR_ERR_INVALID_ARG
    with pytest.raises(B.StarError) as e:                            # listed worker without a buffer
        B.star_group_reduce(out, [grads[0], None, grads[2]], [0, 1])
    assert e.value.status == B.STAR_ERR_NULL_POINTER
    with pytest.raises(B.StarError) as e:
        B.star_group_reduce(out, grads, [0, 1], sum_order=7)
    assert e.value.status == B.STAR_ERR_INVALID_ARG
    B.star_group_reduce(grads[1], grads, [0, 2])                     # an unlisted buffer may be the output
    torch.cuda.synchronize()
    assert B.star_launch_count() == before + 1


@pytest.mark.parametrize("n", [1, 9, 4099, 300_007])
def test_update_from_sums_matches_oracle(B, n):
    gen = torch.Generator(device="cuda").manual_seed(n)
    for R, reports in ((1, 1), (1, 3), (2, 2), (3, 5), (7, 8), (16, 16), (64, 64), (5, 255)):
        p = torch.randn(n, generator=gen, device="cuda") * 0.05
        v = torch.randn(n, generator=gen, device="cuda") * 0.02
        sums = [torch.randn(n, generator=gen, device="cuda") * 0.03 for _ in range(R)]
        p_np, v_np = p.cpu().numpy().copy(), v.cpu().numpy().copy()
        O.update_from_sums_f32(p_np, v_np, [s.cpu().numpy() for s in sums], reports, 0.1, 0.9, 1e-3)
        before = B.star_launch_count()
        B.star_group_update_from_sums(p, v, sums, reports, 0.1, 0.9, 1e-3)
        torch.cuda.synchronize()
        assert B.star_launch_count() == before + 1
        assert_matches(p, p_np, "params R=%d reports=%d" % (R, reports))
        assert_matches(v, v_np, "momentum R=%d reports=%d" % (R, reports))


def test_update_from_sums_errors(B):
    n = 64
    p, v = torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda")
    sums = [torch.ones(n, device="cuda") for _ in range(3)]
    for reports, status in ((2, B.STAR_ERR_INVALID_ARG), (256, B.STAR_ERR_UNSUPPORTED)):
        with pytest.raises(B.StarError) as e:
            B.star_group_update_from_sums(p, v, sums, reports, 0.1, 0.9, 0.0)
        assert e.value.status == status
    with pytest.raises(B.StarError) as e:
        B.star_group_update_from_sums(p, v, [sums[0], p], 2, 0.1, 0.9, 0.0)
    assert e.value.status == B.STAR_ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert not p.any() and not v.any()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_whole_round_equals_the_round_oracle(B, dtype):
    """Nine workers; the three slowest are removed and dealt to parents, one of
    them misses the wait.  Aggregates per ring member, then one update on the
    ring: the GPU composition equals oracle/all_reduce.py bit for bit, and so
    does the single-server form (one group holding the same reports) whenever
    the two orders coincide."""
    n, W = 100_003, 9
    gen = torch.Generator(device="cuda").manual_seed(99)
    p = torch.randn(n, generator=gen, device="cuda") * 0.05
    v = torch.randn(n, generator=gen, device="cuda") * 0.02
    grads = [(torch.randn(n, generator=gen, device="cuda") * 0.01).to(dtype) for _ in range(W)]
    removed, late = [8, 2, 5], [2]
    ring = [w for w in range(W) if w not in removed]
    parent_of = AR.assign_parents(removed, ring)
    in_time = [c for c in removed if c not in late]
    p_np, v_np = p.cpu().numpy().copy(), v.cpu().numpy().copy()
    want_aggr, reports = AR.all_reduce_round_f32(p_np, v_np, [grad_to_numpy(g) for g in grads], ring, parent_of,
                                                 in_time, 0.05, 0.9, 1e-4)
    kids = AR.children_of(parent_of, in_time)
    aggregates = []
    for r in ring:
        a = torch.empty(n, device="cuda")
        B.star_group_reduce(a, grads, [r] + kids.get(r, []))
        aggregates.append(a)
    B.star_group_update_from_sums(p, v, aggregates, reports, 0.05, 0.9, 1e-4)
    torch.cuda.synchronize()
    for a, want in zip(aggregates, want_aggr):
        assert_matches(a, want, "aggregate")
    assert reports == len(ring) + len(in_time) == 8
    assert_matches(p, p_np, "params")
    assert_matches(v, v_np, "momentum")


def test_round_at_the_resnet50_size_every_element(B):
    """An all-reduce round on the ResNet-50-sized workload (8 workers, bf16): two
    workers removed, one in time; every element of the aggregates, p and v."""
    from paper_2512_09685_b200 import workloads as WL
    w = WL.BY_NAME["cfg1_resnet50"]
    n = w.n
    p = WL.make_params(w, "cuda")[0]
    v = WL.make_momentum(w, "cuda")[0]
    grads = [g[0] for g in WL.make_grads(w, 0, "cuda")]
    x, t_w, T, removed, (off, mem) = B.star_choose_all_reduce_mode(
        [1.0, 1.02, 3.0, 0.98, 1.0, 1.05, 5.0, 1.01], [9.0] * 2 + [2.5] + [9.0] * 3 + [1.1, 9.0], 1e4, 256.0, 0.5)
    assert removed == [6, 2] and mem == [0, 1, 3, 4, 5, 6, 7]        # worker 2 misses the wait
    parent_of = B.star_assign_parents(removed, w.W)
    ring = [r for r in range(w.W) if parent_of[r] < 0]
    in_time = [c for c in removed if c in mem]
    p_np, v_np = p.cpu().numpy().copy(), v.cpu().numpy().copy()
    want_aggr, reports = AR.all_reduce_round_f32(p_np, v_np, [grad_to_numpy(g) for g in grads], ring,
                                                 AR.assign_parents(removed, ring), in_time, w.lr, w.mu, w.wd)
    aggregates = []
    for r in ring:
        a = torch.empty(n, device="cuda")
        B.star_group_reduce(a, grads, [r] + sorted(c for c in in_time if parent_of[c] == r))
        aggregates.append(a)
    B.star_group_update_from_sums(p, v, aggregates, reports, w.lr, w.mu, w.wd)
    torch.cuda.synchronize()
    assert reports == 7
    for a, want in zip(aggregates, want_aggr):
        assert_matches(a, want, "aggregate")
    assert_matches(p, p_np, "params")
    assert_matches(v, v_np, "momentum")


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_round_over_a_communication_tree(B, dtype):
    """Section IV-D2b on one GPU: every worker's partial sum (own gradient widened,
    then its children's sums, ascending) with star_group_reduce, the root's sum and
    update with star_group_update_from_sums, against oracle/tree_round.py."""
    from oracle import tree_round as TR
    n, W = 70_003, 11
    gen = torch.Generator(device="cuda").manual_seed(123)
    p = torch.randn(n, generator=gen, device="cuda") * 0.05
    v = torch.randn(n, generator=gen, device="cuda") * 0.02
    grads = [(torch.randn(n, generator=gen, device="cuda") * 0.01).to(dtype) for _ in range(W)]
    for fanout in (1, 2, 3, W):
        latency = [float((7 * w) % W) for w in range(W)]
        parent_of = B.star_build_tree(latency, fanout)
        assert parent_of == TR.build_tree(latency, fanout)
        q, u = p.clone(), v.clone()
        p_np, v_np = p.cpu().numpy().copy(), v.cpu().numpy().copy()
        want_sums = TR.tree_round_f32(p_np, v_np, [grad_to_numpy(g) for g in grads], parent_of, 0.05, 0.9, 1e-4)
        sums = {}

        def partial(w):
            if w not in sums:
                own = torch.empty(n, device="cuda")
                B.star_group_reduce(own, [grads[w]], [0])
                kids = [c for c in range(W) if parent_of[c] == w]
                if kids:
                    total = torch.empty(n, device="cuda")
                    B.star_group_reduce(total, [own] + [partial(c) for c in kids], list(range(len(kids) + 1)))
                    own = total
                sums[w] = own
            return sums[w]
        top = [partial(w) for w in range(W) if parent_of[w] < 0]
        B.star_group_update_from_sums(q, u, top, W, 0.05, 0.9, 1e-4)
        torch.cuda.synchronize()
        for w in range(W):
            assert_matches(partial(w), want_sums[w], "fanout %d partial sum of worker %d" % (fanout, w))
        assert_matches(q, p_np, "fanout %d params" % fanout)
        assert_matches(u, v_np, "fanout %d momentum" % fanout)
