"""The tensor-list path: equal to one call per tensor and to one call on the
concatenation, with ragged sizes, empty tensors and misaligned members."""
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


def build(sizes, W, dtype, seed, misalign=()):
    g = torch.Generator(device="cuda").manual_seed(seed)
    def tensor(s, dt, std, shift):
        raw = torch.empty(s + 3, dtype=dt, device="cuda")
        view = raw[shift: shift + s]
        view.copy_(torch.randn(s, generator=g, device="cuda") * std)
        return view
    params = [tensor(s, torch.float32, 0.05, 1 if t in misalign else 0) for t, s in enumerate(sizes)]
    momentum = [tensor(s, torch.float32, 0.02, 0) for s in sizes]
    grads = [[tensor(s, dtype, 0.01, 0) for s in sizes] for _ in range(W)]
    return params, momentum, grads


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_list_equals_per_tensor_equals_concatenation_equals_oracle(B, dtype):
    W = 5
    params, momentum, grads = build(SIZES, W, dtype, seed=1, misalign=(3, 6))
    off, mem = [0, 2, 3, 5], [3, 0, 4, 1, 2]
    lr, mu, wd = 0.1, 0.9, 1e-3
    # (a) per tensor
    pa = [p.clone() for p in params]
    va = [v.clone() for v in momentum]
    for t, s in enumerate(SIZES):
        B.star_group_update(pa[t], va[t], [grads[w][t] for w in range(W)], off, mem, lr, mu, wd)
    # (b) concatenation
    pc, vc = torch.cat(params), torch.cat(momentum)
    gc = [torch.cat(grads[w]) for w in range(W)]
    # (c) oracle on the concatenation
    p_np, v_np = pc.cpu().numpy().copy(), vc.cpu().numpy().copy()
    O.group_update_f32(p_np, v_np, [grad_to_numpy(g) for g in gc], off, mem, np.float32(lr), mu, wd)
    B.star_group_update(pc, vc, gc, off, mem, lr, mu, wd)
    # (d) the list path, one launch
    ws = torch.empty(B.star_multi_workspace_bytes(SIZES, W), dtype=torch.uint8, device="cuda")
    plan = B.star_multi_prepare(params, momentum, grads, ws)
    assert plan.n_tensors == len(SIZES) and plan.total_elements == sum(SIZES)
    before = B.star_launch_count()
    B.star_group_update_multi(plan, off, mem, lr, mu, wd)
    assert B.star_launch_count() - before == 1
    torch.cuda.synchronize()
    assert torch.equal(torch.cat(params), torch.cat(pa)) and torch.equal(torch.cat(momentum), torch.cat(va))
    assert torch.equal(torch.cat(params), pc) and torch.equal(torch.cat(momentum), vc)
    assert_matches(torch.cat(params), p_np, "params")
    assert_matches(torch.cat(momentum), v_np, "momentum")


def test_plan_is_reusable_across_rounds_with_changing_schedules(B):
    W = 4
    sizes = [5000, 3, 70_001]
    params, momentum, grads = build(sizes, W, torch.bfloat16, seed=2)
    ws = torch.empty(B.star_multi_workspace_bytes(sizes, W) + 512, dtype=torch.uint8, device="cuda")
    plan = B.star_multi_prepare(params, momentum, grads, ws)
    p_np = torch.cat(params).cpu().numpy().copy()
    v_np = torch.cat(momentum).cpu().numpy().copy()
    g_np = [grad_to_numpy(torch.cat(grads[w])) for w in range(W)]
    for off, mem in (([0, 4], [0, 1, 2, 3]), ([0, 1, 2, 3, 4], [3, 2, 1, 0]), ([0, 1, 3], [2, 0, 3])):
        B.star_group_update_multi(plan, off, mem, 0.05, 0.9, 0.01)
        O.group_update_f32(p_np, v_np, g_np, off, mem, np.float32(0.05), 0.9, 0.01)
    torch.cuda.synchronize()
    assert_matches(torch.cat(params), p_np, "params")
    assert_matches(torch.cat(momentum), v_np, "momentum")


def test_list_errors(B):
    W = 3
    sizes = [100, 200]
    params, momentum, grads = build(sizes, W, torch.bfloat16, seed=3)
    need = B.star_multi_workspace_bytes(sizes, W)
    small = torch.empty(need - 1, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.StarError) as e:
        B.star_multi_prepare(params, momentum, grads, small)
    assert e.value.status == B.STAR_ERR_WORKSPACE_TOO_SMALL
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    holes = [list(g) for g in grads]
    holes[2][1] = None                               # worker 2 lacks a gradient for tensor 1
    plan = B.star_multi_prepare(params, momentum, holes, ws)
    p0 = torch.cat(params).clone()
    with pytest.raises(B.StarError) as e:
        B.star_group_update_multi(plan, [0, 3], [0, 1, 2], 0.1, 0.9, 0.0)
    assert e.value.status == B.STAR_ERR_NULL_POINTER
    with pytest.raises(B.StarError) as e:
        B.star_group_update_multi(plan, [0, 0, 2], [0, 1], 0.1, 0.9, 0.0)
    assert e.value.status == B.STAR_ERR_BAD_SCHEDULE
    B.star_group_update_multi(plan, [0, 2], [0, 1], 0.1, 0.9, 0.0)      # workers 0, 1 are complete
    B.star_group_update_multi(plan, [0], [], 0.1, 0.9, 0.0)             # no-op
    torch.cuda.synchronize()
    assert not torch.equal(torch.cat(params), p0)
    empty_plan = B.star_multi_prepare([], [], [[] for _ in range(W)], ws)
    B.star_group_update_multi(empty_plan, [0, 1], [0], 0.1, 0.9, 0.0)


def test_list_round_with_per_group_rates(B):
    W, sizes = 4, [5000, 3, 70_001, 2048]
    params, momentum, grads = build(sizes, W, torch.bfloat16, seed=8)
    ws = torch.empty(B.star_multi_workspace_bytes(sizes, W), dtype=torch.uint8, device="cuda")
    plan = B.star_multi_prepare(params, momentum, grads, ws)
    off, mem, lrs = [0, 1, 4], [2, 0, 1, 3], [0.025, 0.075]
    p_np = torch.cat(params).cpu().numpy().copy()
    v_np = torch.cat(momentum).cpu().numpy().copy()
    g_np = [grad_to_numpy(torch.cat(grads[w])) for w in range(W)]
    O.group_update_f32(p_np, v_np, g_np, off, mem, np.array(lrs, np.float32), 0.9, 0.01)
    B.star_group_update_multi_lrs(plan, off, mem, lrs, 0.9, 0.01)
    torch.cuda.synchronize()
    assert_matches(torch.cat(params), p_np, "params")
    assert_matches(torch.cat(momentum), v_np, "momentum")
    with pytest.raises(ValueError):
        B.star_group_update_multi_lrs(plan, off, mem, [0.1], 0.9, 0.01)


def test_aliased_list_entries_are_refused(B):
    """A buffer that a round writes may not share memory with any other buffer
    of the list, in whichever tensor: different blocks would update it at once."""
    W, sizes = 2, [1000, 1000, 64]
    params, momentum, grads = build(sizes, W, torch.bfloat16, seed=4)
    ws = torch.empty(B.star_multi_workspace_bytes(sizes, W), dtype=torch.uint8, device="cuda")
    before = B.star_launch_count()
    tied = list(params)
    tied[1] = params[0]                               # a tied weight listed twice
    crossed = list(momentum)
    crossed[1] = params[0]                            # one tensor's momentum is another's parameters
    for bad_p, bad_v in ((tied, momentum), (params, crossed)):
        with pytest.raises(B.StarError) as e:
            B.star_multi_prepare(bad_p, bad_v, grads, ws)
        assert e.value.status == B.STAR_ERR_INVALID_ARG
    read_only = [[torch.zeros(s, dtype=torch.bfloat16, device="cuda") for s in sizes]] * W
    B.star_multi_prepare(params, momentum, read_only, ws)          # gradients may alias one another
    written = [list(g) for g in grads]
    written[1][2] = params[0].view(torch.bfloat16)[:64]             # a gradient inside another tensor's parameters
    with pytest.raises(B.StarError) as e:
        B.star_multi_prepare(params, momentum, written, ws)
    assert e.value.status == B.STAR_ERR_INVALID_ARG
    assert B.star_launch_count() == before


def test_prepare_refuses_to_run_inside_a_stream_capture(B):
    """The table is copied from host memory that is released on return; a graph
    would read it again at every replay.  The call says so and enqueues nothing;
    the capture is ended and the graph is never replayed."""
    W, sizes = 2, [300, 5000]
    params, momentum, grads = build(sizes, W, torch.bfloat16, seed=5)
    ws = torch.zeros(B.star_multi_workspace_bytes(sizes, W), dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    status = None
    with torch.cuda.stream(side):
        graph.capture_begin()
        try:
            B.star_multi_prepare(params, momentum, grads, ws, stream=side)
        except B.StarError as e:
            status = e.status
        graph.capture_end()
    torch.cuda.synchronize()
    assert status == B.STAR_ERR_UNSUPPORTED
    assert not ws.any()                                # nothing was copied
    del graph
