"""The allocation-free tensor-list entry point against the workspace-based one.

Collected last on purpose (file name): if it fails, a run that stops at the
first failure has already run every other test.

Who needs it: code that cannot get device memory at call time -- a plug-in
running after its host framework's pool has taken all free memory, a hook on a
path where cudaMalloc's device-wide synchronization is not acceptable, or
start-up code that runs before any allocator exists.  Such callers still pass
their own parameter, momentum and gradient buffers; only the pointer table
moves into a fixed array inside the library, shared by all calls on a device.
This test therefore runs two different lists back to back (the second smaller
than the first, so stale table entries lie behind it) and checks both against
the ordinary prepare + update path, bit for bit.
"""
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2512_09685_b200 import binding
    return binding


def make_list(sizes, W, dtype, seed):
    g = torch.Generator(device="cuda").manual_seed(seed)
    params = [torch.randn(s, generator=g, device="cuda") * 0.05 for s in sizes]
    momentum = [torch.randn(s, generator=g, device="cuda") * 0.02 for s in sizes]
    grads = [[(torch.randn(s, generator=g, device="cuda") * 0.01).to(dtype) for s in sizes]
             for _ in range(W)]
    return params, momentum, grads


def reference(B, params, momentum, grads, off, mem, lr, mu, wd):
    """The existing entry points on clones, with a caller-provided workspace."""
    p = [x.clone() for x in params]
    v = [x.clone() for x in momentum]
    sizes = [x.numel() for x in p]
    ws = torch.empty(B.star_multi_workspace_bytes(sizes, len(grads)), dtype=torch.uint8, device="cuda")
    plan = B.star_multi_prepare(p, v, grads, ws)
    B.star_group_update_multi(plan, off, mem, lr, mu, wd)
    torch.cuda.synchronize()
    return p, v


def same_bits(xs, ys):
    return all(torch.equal(x.view(torch.int32), y.view(torch.int32)) for x, y in zip(xs, ys))


def test_two_calls_in_a_row_match_the_workspace_path(B):
    cases = [
        # a larger list first ...
        ([70_001, 5, 0, 4096, 33, 262_144, 2048, 1], 6, torch.bfloat16,
         ([0, 2, 3, 6], [5, 1, 0, 2, 3, 4]), (0.1, 0.9, 1e-3)),
        # ... then a smaller one with another dtype, width and schedule
        ([1000, 17, 40_000], 3, torch.float32, ([0, 1, 2], [2, 0]), (0.05, 0.8, 0.0)),
    ]
    for call, (sizes, W, dtype, (off, mem), (lr, mu, wd)) in enumerate(cases):
        params, momentum, grads = make_list(sizes, W, dtype, seed=100 + call)
        want_p, want_v = reference(B, params, momentum, grads, off, mem, lr, mu, wd)
        p0 = [x.clone() for x in params]
        launches = B.star_launch_count()
        B.star_group_update_multi_noalloc(params, momentum, grads, off, mem, lr, mu, wd)
        torch.cuda.synchronize()
        assert B.star_launch_count() == launches + 1
        assert same_bits(params, want_p), "call %d params" % call
        assert same_bits(momentum, want_v), "call %d momentum" % call
        assert not same_bits([params[0]], [p0[0]])            # it did update


def test_repeated_rounds_on_one_list_and_on_a_side_stream(B):
    sizes, W = [12_345, 8, 50_000], 4
    params, momentum, grads = make_list(sizes, W, torch.bfloat16, seed=7)
    p_ref = [x.clone() for x in params]
    v_ref = [x.clone() for x in momentum]
    ws = torch.empty(B.star_multi_workspace_bytes(sizes, W), dtype=torch.uint8, device="cuda")
    plan = B.star_multi_prepare(p_ref, v_ref, grads, ws)
    schedules = [([0, 4], [0, 1, 2, 3]), ([0, 1, 2, 3, 4], [3, 1, 0, 2]), ([0, 2, 3], [1, 3, 0])]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    for off, mem in schedules:
        B.star_group_update_multi(plan, off, mem, 0.1, 0.9, 1e-4)
        with torch.cuda.stream(side):                          # same stream every time: ordered
            B.star_group_update_multi_noalloc(params, momentum, grads, off, mem, 0.1, 0.9, 1e-4)
    torch.cuda.synchronize()
    assert same_bits(params, p_ref) and same_bits(momentum, v_ref)


def test_limits_and_errors(B):
    # a table larger than the fixed array is refused, and nothing is touched
    W = 2
    n_tensors = B.STAR_STATIC_SCRATCH_BYTES // 40 + 1          # entries alone exceed the array
    shared_p = torch.zeros(4, device="cuda")
    shared_v = torch.zeros(4, device="cuda")
    g = torch.ones(4, device="cuda")
    sizes_need = B.star_multi_workspace_bytes([4] * n_tensors, W)
    assert sizes_need > B.STAR_STATIC_SCRATCH_BYTES
    # distinct views are not needed to hit the size check, which comes first
    with pytest.raises(B.StarError) as e:
        B.star_group_update_multi_noalloc([shared_p] * n_tensors, [shared_v] * n_tensors,
                                          [[g] * n_tensors] * W, [0, 1], [0], 0.1, 0.9, 0.0)
    assert e.value.status == B.STAR_ERR_WORKSPACE_TOO_SMALL
    assert float(shared_p.abs().sum()) == 0.0
    params, momentum, grads = make_list([100, 200], W, torch.bfloat16, seed=9)
    p0 = [x.clone() for x in params]
    with pytest.raises(B.StarError) as e:
        B.star_group_update_multi_noalloc(params, momentum, grads, [0, 0, 2], [0, 1], 0.1, 0.9, 0.0)
    assert e.value.status == B.STAR_ERR_BAD_SCHEDULE
    B.star_group_update_multi_noalloc(params, momentum, grads, [0], [], 0.1, 0.9, 0.0)     # no-op
    torch.cuda.synchronize()
    assert same_bits(params, p0)


def test_refused_inside_a_stream_capture(B):
    """Called while its stream is being captured the entry point returns
    STAR_ERR_UNSUPPORTED before it touches the shared table or the caller's
    tensors; the capture is ended and the graph is never replayed.  A normal
    call afterwards still matches the workspace path."""
    sizes, W = [4000, 9, 30_000], 3
    params, momentum, grads = make_list(sizes, W, torch.bfloat16, seed=11)
    off, mem = [0, 2, 3], [2, 0, 1]
    B.star_group_update_multi_noalloc(params, momentum, grads, off, mem, 0.1, 0.9, 1e-4)   # set-up outside capture
    torch.cuda.synchronize()
    p0 = [x.clone() for x in params]
    launches = B.star_launch_count()
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    status = None
    with torch.cuda.stream(side):
        graph.capture_begin()
        try:
            B.star_group_update_multi_noalloc(params, momentum, grads, off, mem, 0.1, 0.9, 1e-4, stream=side)
        except B.StarError as e:
            status = e.status
        graph.capture_end()
    torch.cuda.synchronize()
    del graph
    assert status == B.STAR_ERR_UNSUPPORTED
    assert B.star_launch_count() == launches
    assert same_bits(params, p0)
    want_p, want_v = reference(B, params, momentum, grads, off, mem, 0.1, 0.9, 1e-4)
    B.star_group_update_multi_noalloc(params, momentum, grads, off, mem, 0.1, 0.9, 1e-4)
    torch.cuda.synchronize()
    assert same_bits(params, want_p) and same_bits(momentum, want_v)


def test_error_found_after_the_table_was_rewritten(B):
    """Scheduling a worker that has no gradient for some tensor is only seen once
    the table is in place: nothing is launched, the tensors stay as they were,
    and the next good call is still right."""
    sizes, W = [700, 4096], 3
    params, momentum, grads = make_list(sizes, W, torch.float32, seed=12)
    holes = [list(g) for g in grads]
    holes[2][1] = None
    p0 = [x.clone() for x in params]
    launches = B.star_launch_count()
    with pytest.raises(B.StarError) as e:
        B.star_group_update_multi_noalloc(params, momentum, holes, [0, 3], [0, 1, 2], 0.1, 0.9, 0.0)
    assert e.value.status == B.STAR_ERR_NULL_POINTER
    torch.cuda.synchronize()
    assert B.star_launch_count() == launches and same_bits(params, p0)
    want_p, want_v = reference(B, params, momentum, holes, [0, 2], [1, 0], 0.1, 0.9, 0.0)
    B.star_group_update_multi_noalloc(params, momentum, holes, [0, 2], [1, 0], 0.1, 0.9, 0.0)
    B.star_group_update_multi_noalloc([], [], [[] for _ in range(W)], [0, 1], [0], 0.1, 0.9, 0.0)   # empty list
    torch.cuda.synchronize()
    assert same_bits(params, want_p) and same_bits(momentum, want_v)


def test_a_list_that_fills_the_fixed_array_exactly(B):
    """The largest list that still fits: its table needs exactly STAR_STATIC_SCRATCH_BYTES."""
    W = 1
    n_tensors = 1
    while B.star_multi_workspace_bytes([8] * (n_tensors + 1), W) <= B.STAR_STATIC_SCRATCH_BYTES:
        n_tensors += 1
    # pad the last step with larger tensors until the table size lands on the limit
    sizes = [8] * n_tensors
    assert B.star_multi_workspace_bytes(sizes, W) <= B.STAR_STATIC_SCRATCH_BYTES
    grow = 0
    while B.star_multi_workspace_bytes(sizes, W) < B.STAR_STATIC_SCRATCH_BYTES and grow < n_tensors:
        sizes[grow] = 1024 * 64 + 8                      # 64 more tiles' worth of map entries
        grow += 1
    assert B.star_multi_workspace_bytes(sizes, W) == B.STAR_STATIC_SCRATCH_BYTES
    g = torch.Generator(device="cuda").manual_seed(13)
    flat_p = torch.randn(sum(sizes), generator=g, device="cuda") * 0.05
    flat_v = torch.zeros(sum(sizes), device="cuda")
    flat_g = torch.randn(sum(sizes), generator=g, device="cuda") * 0.01
    params, momentum, grads = list(flat_p.split(sizes)), list(flat_v.split(sizes)), [list(flat_g.split(sizes))]
    want_p = flat_p.clone()
    want_v = flat_v.clone()
    B.star_group_update(want_p, want_v, [flat_g], [0, 1], [0], 0.1, 0.9, 1e-4)
    B.star_group_update_multi_noalloc(params, momentum, grads, [0, 1], [0], 0.1, 0.9, 1e-4)
    torch.cuda.synchronize()
    assert torch.equal(flat_p, want_p) and torch.equal(flat_v, want_v)
