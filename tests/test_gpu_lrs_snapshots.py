"""Per-group learning rates and parameter snapshots (the copy sent back to a
group's workers) in the fused kernel, against the oracle and closed forms."""
import numpy as np
import pytest
import torch

from oracle import schedule as S
from oracle import star_oracle as O
from tests.parity import assert_matches, grad_to_numpy

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2512_09685_b200 import binding
    return binding


def case(n, W, dtype, seed):
    g = torch.Generator(device="cuda").manual_seed(seed)
    p = torch.randn(n, generator=g, device="cuda") * 0.05
    v = torch.randn(n, generator=g, device="cuda") * 0.02
    grads = [(torch.randn(n, generator=g, device="cuda") * 0.01).to(dtype) for _ in range(W)]
    return p, v, grads


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("n", [1, 7, 4099, 1_000_003])
def test_lrs_and_snapshots_match_oracle(B, dtype, n):
    W = 8
    p, v, grads = case(n, W, dtype, seed=n)
    off, mem = [0, 3, 4, 6, 8], [5, 0, 2, 7, 1, 3, 4, 6]
    lrs = [0.1, 0.025, 0.05, 0.2]
    p_np, v_np = p.cpu().numpy().copy(), v.cpu().numpy().copy()
    g_np = [grad_to_numpy(g) for g in grads]
    want_snaps = [np.zeros(n, np.float32), None, np.zeros(n, np.float32), np.zeros(n, np.float32)]
    O.group_update_f32(p_np, v_np, g_np, off, mem, np.array(lrs, np.float32), 0.9, 1e-3, snapshots=want_snaps)
    snaps = [torch.full((n,), float("nan"), device="cuda"), None,
             torch.full((n,), float("nan"), device="cuda"), torch.full((n,), float("nan"), device="cuda")]
    before = B.star_launch_count()
    B.star_group_update_ex(p, v, grads, off, mem, lrs, 0.9, 1e-3, snapshots=snaps)
    torch.cuda.synchronize()
    assert B.star_launch_count() == before + 1
    assert_matches(p, p_np, "params")
    assert_matches(v, v_np, "momentum")
    for k in (0, 2, 3):
        assert_matches(snaps[k], want_snaps[k], "snapshot %d" % k)
    assert torch.equal(snaps[3], p)                    # the last group's snapshot is the final state


def test_misaligned_snapshot_takes_the_scalar_path(B):
    n = 5001
    p, v, grads = case(n, 3, torch.bfloat16, seed=2)
    p_np, v_np = p.cpu().numpy().copy(), v.cpu().numpy().copy()
    want = [np.zeros(n, np.float32), None]
    O.group_update_f32(p_np, v_np, [grad_to_numpy(g) for g in grads], [0, 2, 3], [0, 1, 2],
                       np.array([0.1, 0.2], np.float32), 0.9, 0.0, snapshots=want)
    snap = torch.empty(n + 1, device="cuda")[1:]
    B.star_group_update_ex(p, v, grads, [0, 2, 3], [0, 1, 2], [0.1, 0.2], 0.9, 0.0, snapshots=[snap, None])
    torch.cuda.synchronize()
    assert_matches(p, p_np, "params")
    assert_matches(snap, want[0], "snapshot")


def test_equal_rates_without_snapshots_equal_the_plain_entry_point(B):
    n = 77_777
    p, v, grads = case(n, 6, torch.bfloat16, seed=3)
    q, u = p.clone(), v.clone()
    off, mem = [0, 2, 6], [1, 0, 5, 4, 3, 2]
    B.star_group_update(p, v, grads, off, mem, 0.05, 0.9, 1e-4)
    B.star_group_update_ex(q, u, grads, off, mem, [0.05, 0.05], 0.9, 1e-4)
    torch.cuda.synchronize()
    assert torch.equal(p, q) and torch.equal(v, u)


def test_rescaled_rates_make_the_round_schedule_independent(B):
    """Section IV-C1: r_new = (y / N) r_SSGD.  With mu = wd = 0 every covering
    schedule then lands on p0 - (r / N) sum_w g_w (up to fp32 rounding)."""
    n, N, r = 50_000, 8, 0.4
    p0, _, grads = case(n, N, torch.float32, seed=4)
    want = p0.double() - (r / N) * sum(g.double() for g in grads)
    for x in (1, 2, 3, 4, 8):
        off, mem = B.star_schedule_static_x(None, N, x)
        lrs = S.scaled_lrs(off, len(off) - 1, N, r)
        p, v = p0.clone(), torch.zeros(n, device="cuda")
        B.star_group_update_ex(p, v, grads, off, mem, lrs, 0.0, 0.0)
        torch.cuda.synchronize()
        assert float((p.double() - want).abs().max()) <= 16 * 2.0 ** -24 * float(want.abs().max())


def test_ex_errors(B):
    n = 1000
    p, v, grads = case(n, 2, torch.bfloat16, seed=5)
    p0 = p.clone()
    with pytest.raises(B.StarError) as e:              # snapshot overlaps params
        B.star_group_update_ex(p, v, grads, [0, 2], [0, 1], [0.1], 0.9, 0.0, snapshots=[p])
    assert e.value.status == B.STAR_ERR_INVALID_ARG
    s = torch.empty(n, device="cuda")
    with pytest.raises(B.StarError) as e:              # two groups into one buffer
        B.star_group_update_ex(p, v, grads, [0, 1, 2], [0, 1], [0.1, 0.1], 0.9, 0.0, snapshots=[s, s])
    assert e.value.status == B.STAR_ERR_INVALID_ARG
    with pytest.raises(ValueError):
        B.star_group_update_ex(p, v, grads, [0, 1, 2], [0, 1], [0.1], 0.9, 0.0)
    torch.cuda.synchronize()
    assert torch.equal(p, p0)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_tree_summation_order_matches_oracle(B, dtype):
    """Group sizes 1..9, 16, 17, 33, 64 in the pairwise (aggregation tree) order."""
    rng = np.random.default_rng(7)
    for size in list(range(1, 10)) + [16, 17, 33, 64]:
        W = min(64, size + 2)
        for n in (5, 4099, 200_003):
            p, v, grads = case(n, W, dtype, seed=size * 7 + n)
            members = [int(w) for w in rng.permutation(W)[:size]]
            if size >= 3:
                off, mem = [0, size - 1, size], members
            else:
                off, mem = [0, size], members
            lrs = [0.1] * (len(off) - 1)
            p_np, v_np = p.cpu().numpy().copy(), v.cpu().numpy().copy()
            g_np = [grad_to_numpy(g) for g in grads]
            want_snap = [np.zeros(n, np.float32)] + [None] * (len(off) - 2)
            O.group_update_f32(p_np, v_np, g_np, off, mem, np.array(lrs, np.float32), 0.9, 1e-3,
                               snapshots=want_snap, sum_order="tree")
            snap = [torch.empty(n, device="cuda")] + [None] * (len(off) - 2)
            B.star_group_update_ex(p, v, grads, off, mem, lrs, 0.9, 1e-3, snapshots=snap,
                                   sum_order=B.STAR_SUM_TREE)
            torch.cuda.synchronize()
            assert_matches(p, p_np, "params size=%d n=%d" % (size, n))
            assert_matches(v, v_np, "momentum size=%d n=%d" % (size, n))
            assert_matches(snap[0], want_snap[0], "snapshot size=%d n=%d" % (size, n))


def test_tree_and_linear_orders_differ_only_in_rounding(B):
    n = 100_000
    p, v, grads = case(n, 9, torch.float32, seed=11)
    q, u = p.clone(), v.clone()
    off, mem = [0, 9], list(range(9))
    B.star_group_update_ex(p, v, grads, off, mem, [0.1], 0.9, 1e-4, sum_order=B.STAR_SUM_LINEAR)
    B.star_group_update_ex(q, u, grads, off, mem, [0.1], 0.9, 1e-4, sum_order=B.STAR_SUM_TREE)
    torch.cuda.synchronize()
    assert not torch.equal(p, q)
    assert float((p - q).abs().max()) <= 8 * 2.0 ** -24 * 0.1
    with pytest.raises(B.StarError):
        B.star_group_update_ex(p, v, grads, off, mem, [0.1], 0.9, 1e-4, sum_order=5)


@pytest.mark.parametrize("n", [3, 4099, 500_001])
def test_bf16_snapshots_match_oracle(B, n):
    W = 6
    p, v, grads = case(n, W, torch.bfloat16, seed=n + 1)
    # plant exact ties for the narrowing in the first snapshot: p' = p - lr * v' with v' = g, lr = 1
    off, mem = [0, 2, 6], [1, 0, 5, 4, 3, 2]
    p_np, v_np = p.cpu().numpy().copy(), v.cpu().numpy().copy()
    g_np = [grad_to_numpy(g) for g in grads]
    want = [np.zeros(n, np.uint16), np.zeros(n, np.uint16)]
    O.group_update_f32(p_np, v_np, g_np, off, mem, np.array([0.1, 0.05], np.float32), 0.9, 1e-3, snapshots=want)
    snaps = [torch.zeros(n, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    B.star_group_update_ex(p, v, grads, off, mem, [0.1, 0.05], 0.9, 1e-3, snapshots=snaps)
    torch.cuda.synchronize()
    assert_matches(p, p_np, "params")
    for k in range(2):
        got = snaps[k].cpu().view(torch.int16).numpy().view(np.uint16)
        assert np.array_equal(got, want[k]), "snapshot %d" % k
    assert torch.equal(snaps[1], p.to(torch.bfloat16))            # torch's cast rounds the same way


def test_bf16_snapshot_narrowing_on_ties_and_extremes(B):
    """Zero gradients and momentum hold the parameters still: the snapshot is the
    narrowing of the input, compared with the oracle and with torch's cast."""
    from tests.test_oracle_pins import bf16_snapshot_probe_values
    x = bf16_snapshot_probe_values()
    n = x.size
    p = torch.from_numpy(x.copy()).cuda()
    v = torch.zeros(n, device="cuda")
    g = torch.zeros(n, device="cuda")
    for misalign in (0, 1):
        raw = torch.zeros(n + 1, dtype=torch.bfloat16, device="cuda")
        snap = raw[misalign: misalign + n]
        B.star_group_update_ex(p, v, [g], [0, 1], [0], [0.1], 0.9, 0.0, snapshots=[snap])
        torch.cuda.synchronize()
        assert torch.equal(snap.view(torch.int16), torch.from_numpy(x).cuda().to(torch.bfloat16).view(torch.int16))
    want = np.zeros(n, np.uint16)
    O.group_update_f32(x.copy(), np.zeros(n, np.float32), [np.zeros(n, np.float32)], [0, 1], [0], 0.1, 0.9, 0.0,
                       snapshots=[want])
    assert np.array_equal(snap.cpu().view(torch.int16).numpy().view(np.uint16), want)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("snap_dtype", [torch.float32, torch.bfloat16])
def test_views_at_a_common_element_offset(B, dtype, snap_dtype):
    """Every buffer a view at the same odd element offset into aligned storage
    (vector body behind a few leading elements), and one with the snapshot
    out of phase (element path): same bits as the oracle, guard bands intact."""
    pad = 32
    for offset in (1, 3, 7, 8, 9, 13):
        for n in (2, 9, 4099, 70_001):
            for snap_extra in (0, 1):
                g = torch.Generator(device="cuda").manual_seed(offset * 1000 + n)

                def carve(dt, std, shift):
                    raw = torch.full((n + 2 * pad + shift,), float("nan"), dtype=dt, device="cuda")
                    view = raw[pad + shift: pad + shift + n]
                    view.copy_(torch.randn(n, generator=g, device="cuda") * std)
                    return raw, view
                (p_raw, p), (v_raw, v) = carve(torch.float32, 0.05, offset), carve(torch.float32, 0.02, offset)
                grads = [carve(dtype, 0.01, offset)[1] for _ in range(6)]
                s_raw, snap = carve(snap_dtype, 0.0, offset + snap_extra)
                off, mem, lrs = [0, 5, 6], [4, 0, 5, 2, 1, 3], [0.1, 0.05]
                for order, name in ((B.STAR_SUM_LINEAR, "linear"), (B.STAR_SUM_TREE, "tree")):
                    q, u = p.clone(), v.clone()
                    p_np, v_np = p.cpu().numpy().copy(), v.cpu().numpy().copy()
                    want = [np.zeros(n, np.uint16 if snap_dtype == torch.bfloat16 else np.float32), None]
                    O.group_update_f32(p_np, v_np, [grad_to_numpy(x) for x in grads], off, mem,
                                       np.array(lrs, np.float32), 0.9, 1e-3, snapshots=want, sum_order=name)
                    B.star_group_update_ex(p, v, grads, off, mem, lrs, 0.9, 1e-3, snapshots=[snap, None],
                                           sum_order=order)
                    torch.cuda.synchronize()
                    what = "offset=%d n=%d extra=%d %s" % (offset, n, snap_extra, name)
                    assert_matches(p, p_np, "params " + what)
                    assert_matches(v, v_np, "momentum " + what)
                    if snap_dtype == torch.bfloat16:
                        assert np.array_equal(snap.cpu().view(torch.int16).numpy().view(np.uint16), want[0]), what
                    else:
                        assert_matches(snap, want[0], "snapshot " + what)
                    for raw, shift in ((p_raw, offset), (v_raw, offset), (s_raw, offset + snap_extra)):
                        assert bool(torch.isnan(raw[: pad + shift].float()).all()), what
                        assert bool(torch.isnan(raw[pad + shift + n:].float()).all()), what
                    p.copy_(q)
                    v.copy_(u)
