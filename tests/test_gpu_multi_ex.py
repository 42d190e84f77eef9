"""Tensor lists with per-group rates, parameter snapshots (Section II: the copy
sent back to a group's workers) and the tree order (Section IV-D2b) in one
launch: against the oracle on the concatenation and against the flat extended
entry point tensor by tensor."""
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


SIZES = [1, 0, 7, 4096, 4097, 15, 33_000, 8, 2048, 0, 100_003, 16, 31, 262_144, 5]


def build(sizes, W, dtype, seed, shift_of=lambda t: 0):
    """Every buffer of tensor t is a view at shift_of(t) elements into its own
    allocation: a common phase per tensor, different between tensors."""
    g = torch.Generator(device="cuda").manual_seed(seed)

    def tensor(s, dt, std, shift):
        raw = torch.empty(s + 16, dtype=dt, device="cuda")
        view = raw[shift: shift + s]
        view.copy_(torch.randn(s, generator=g, device="cuda") * std)
        return view
    params = [tensor(s, torch.float32, 0.05, shift_of(t)) for t, s in enumerate(sizes)]
    momentum = [tensor(s, torch.float32, 0.02, shift_of(t)) for t, s in enumerate(sizes)]
    grads = [[tensor(s, dtype, 0.01, shift_of(t)) for t, s in enumerate(sizes)] for _ in range(W)]
    return params, momentum, grads


def snapshot_sets(sizes, n_sets, dtype, shift_of=lambda t: 0):
    out = []
    for _ in range(n_sets):
        one = []
        for t, s in enumerate(sizes):
            raw = torch.full((s + 16,), float("nan"), dtype=dtype, device="cuda")
            one.append(raw[shift_of(t): shift_of(t) + s])
        out.append(one)
    return out


def bits(t):
    return t.cpu().view(torch.int16).numpy().view(np.uint16)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("snap_dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("order", ["linear", "tree"])
def test_list_with_snapshots_matches_oracle_and_the_flat_entry_point(B, dtype, snap_dtype, order):
    W = 9
    shift = lambda t: t % 9                                     # noqa: E731  (phases 0..8 elements)
    params, momentum, grads = build(SIZES, W, dtype, seed=21, shift_of=shift)
    sets = snapshot_sets(SIZES, 2, snap_dtype, shift_of=shift)
    sets[1][6] = None                                           # set 1 does not capture tensor 6
    off, mem = [0, 5, 6, 9], [3, 0, 4, 8, 6, 1, 2, 7, 5]       # a group of 5: the tree order differs
    lrs = [0.1, 0.025, 0.05]
    set_of_group = [1, -1, 0]
    sum_order = B.STAR_SUM_TREE if order == "tree" else B.STAR_SUM_LINEAR

    # oracle on the concatenation
    p_np = torch.cat(params).cpu().numpy().copy()
    v_np = torch.cat(momentum).cpu().numpy().copy()
    g_np = [grad_to_numpy(torch.cat(grads[w])) for w in range(W)]
    n = p_np.size
    snap_np = np.uint16 if snap_dtype == torch.bfloat16 else np.float32
    want_snaps = [np.zeros(n, snap_np), None, np.zeros(n, snap_np)]
    O.group_update_f32(p_np, v_np, g_np, off, mem, np.array(lrs, np.float32), 0.9, 1e-3, snapshots=want_snaps,
                       sum_order=order)

    # flat extended entry point, tensor by tensor, on clones
    pa, va = [p.clone() for p in params], [v.clone() for v in momentum]
    for t, s in enumerate(SIZES):
        B.star_group_update_ex(pa[t], va[t], [grads[w][t] for w in range(W)], off, mem, lrs, 0.9, 1e-3,
                               sum_order=sum_order)

    ws = torch.empty(B.star_multi_workspace_bytes_ex(SIZES, W, 2), dtype=torch.uint8, device="cuda")
    plan = B.star_multi_prepare_ex(params, momentum, grads, sets, ws)
    assert plan.n_snapshot_sets == 2
    before = B.star_launch_count()
    B.star_group_update_multi_ex(plan, off, mem, lrs, 0.9, 1e-3, set_of_group, sum_order)
    assert B.star_launch_count() == before + 1
    torch.cuda.synchronize()
    assert torch.equal(torch.cat(params), torch.cat(pa)) and torch.equal(torch.cat(momentum), torch.cat(va))
    assert_matches(torch.cat(params), p_np, "params")
    assert_matches(torch.cat(momentum), v_np, "momentum")
    starts = np.concatenate([[0], np.cumsum(SIZES)])
    for k, set_index in enumerate(set_of_group):
        if set_index < 0:
            continue
        for t, s in enumerate(SIZES):
            buf = sets[set_index][t]
            if buf is None or s == 0:
                continue
            want = want_snaps[k][starts[t]: starts[t + 1]]
            if snap_dtype == torch.bfloat16:
                assert np.array_equal(bits(buf), want), "snapshot of group %d tensor %d" % (k, t)
            else:
                assert_matches(buf, want, "snapshot of group %d tensor %d" % (k, t))


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_list_tree_order_for_every_kernel_variant(B, dtype):
    """Groups of 3, 4, 9, 16, 17, 40 and 64 members through the list kernels."""
    sizes = [5, 4099, 70_001, 2048]
    rng = np.random.default_rng(5)
    for size in (3, 4, 9, 16, 17, 40, 64):
        W = min(64, size + 2)
        params, momentum, grads = build(sizes, W, dtype, seed=size, shift_of=lambda t: 3 * t)
        members = [int(w) for w in rng.permutation(W)[:size]]
        off, mem = [0, size - 1, size], members
        p_np = torch.cat(params).cpu().numpy().copy()
        v_np = torch.cat(momentum).cpu().numpy().copy()
        g_np = [grad_to_numpy(torch.cat(grads[w])) for w in range(W)]
        O.group_update_f32(p_np, v_np, g_np, off, mem, np.array([0.1, 0.2], np.float32), 0.9, 1e-3,
                           sum_order="tree")
        ws = torch.empty(B.star_multi_workspace_bytes(sizes, W), dtype=torch.uint8, device="cuda")
        plan = B.star_multi_prepare(params, momentum, grads, ws)
        B.star_group_update_multi_ex(plan, off, mem, [0.1, 0.2], 0.9, 1e-3, None, B.STAR_SUM_TREE)
        torch.cuda.synchronize()
        assert_matches(torch.cat(params), p_np, "params size=%d" % size)
        assert_matches(torch.cat(momentum), v_np, "momentum size=%d" % size)


def test_plain_rounds_on_a_plan_with_snapshot_sets_and_changing_choices(B):
    W, sizes = 4, [5000, 3, 70_001]
    params, momentum, grads = build(sizes, W, torch.bfloat16, seed=2)
    sets = snapshot_sets(sizes, 3, torch.float32)
    ws = torch.empty(B.star_multi_workspace_bytes_ex(sizes, W, 3), dtype=torch.uint8, device="cuda")
    plan = B.star_multi_prepare_ex(params, momentum, grads, sets, ws)
    p_np = torch.cat(params).cpu().numpy().copy()
    v_np = torch.cat(momentum).cpu().numpy().copy()
    g_np = [grad_to_numpy(torch.cat(grads[w])) for w in range(W)]
    n = p_np.size
    # round 1: plain entry point on the same plan; round 2: two groups into sets 2 and 0
    B.star_group_update_multi(plan, [0, 4], [0, 1, 2, 3], 0.05, 0.9, 0.01)
    O.group_update_f32(p_np, v_np, g_np, [0, 4], [0, 1, 2, 3], np.float32(0.05), 0.9, 0.01)
    want = [np.zeros(n, np.float32), np.zeros(n, np.float32)]
    B.star_group_update_multi_ex(plan, [0, 1, 4], [3, 2, 1, 0], [0.05, 0.1], 0.9, 0.01, [2, 0])
    O.group_update_f32(p_np, v_np, g_np, [0, 1, 4], [3, 2, 1, 0], np.array([0.05, 0.1], np.float32), 0.9, 0.01,
                       snapshots=want)
    torch.cuda.synchronize()
    assert_matches(torch.cat(params), p_np, "params")
    assert_matches(torch.cat(sets[2]), want[0], "set 2")
    assert_matches(torch.cat(sets[0]), want[1], "set 0")
    assert bool(torch.isnan(torch.cat(sets[1])).all())          # set 1 was never chosen


def test_ex_list_errors(B):
    W, sizes = 3, [100, 200]
    params, momentum, grads = build(sizes, W, torch.bfloat16, seed=3)
    sets = snapshot_sets(sizes, 1, torch.float32)
    ws = torch.empty(B.star_multi_workspace_bytes_ex(sizes, W, 1), dtype=torch.uint8, device="cuda")
    plan = B.star_multi_prepare_ex(params, momentum, grads, sets, ws)
    p0 = torch.cat(params).clone()
    for choice in ([1, -1], [-2, 0]):
        with pytest.raises(B.StarError) as e:                   # set index out of range
            B.star_group_update_multi_ex(plan, [0, 1, 2], [0, 1], [0.1, 0.1], 0.9, 0.0, choice)
        assert e.value.status == B.STAR_ERR_INVALID_ARG
    with pytest.raises(B.StarError) as e:
        B.star_group_update_multi_ex(plan, [0, 1, 2], [0, 1], [0.1, 0.1], 0.9, 0.0, None, 9)
    assert e.value.status == B.STAR_ERR_INVALID_ARG
    # a snapshot buffer that is also a parameter buffer of another tensor is refused at prepare time
    bad = [[params[1][:100], None]]
    with pytest.raises(B.StarError) as e:
        B.star_multi_prepare_ex(params, momentum, grads, bad, ws)
    assert e.value.status == B.STAR_ERR_INVALID_ARG
    small = torch.empty(B.star_multi_workspace_bytes_ex(sizes, W, 1) - 1, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.StarError) as e:
        B.star_multi_prepare_ex(params, momentum, grads, sets, small)
    assert e.value.status == B.STAR_ERR_WORKSPACE_TOO_SMALL
    torch.cuda.synchronize()
    assert torch.equal(torch.cat(params), p0)
