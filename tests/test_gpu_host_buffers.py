"""The host-buffer entry point: chunked streaming through a device workspace
gives the oracle's result on host tensors, for pinned and pageable memory,
several chunk sizes, ragged tails and partial schedules."""
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


def host_case(n, W, dtype, seed, pinned):
    g = torch.Generator().manual_seed(seed)
    mk = lambda dt, std: (torch.randn(n, generator=g) * std).to(dt)
    tensors = [mk(torch.float32, 0.05), mk(torch.float32, 0.02)] + [mk(dtype, 0.01) for _ in range(W)]
    if pinned:
        tensors = [t.pin_memory() for t in tensors]
    return tensors[0], tensors[1], tensors[2:]


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("pinned", [True, False])
def test_host_update_matches_oracle_over_many_chunks(B, dtype, pinned):
    n, W = 1_000_003, 6
    off, mem = [0, 2, 3, 5], [4, 0, 2, 5, 1]                  # worker 3 unscheduled
    for chunk in (2048, 65536, 4 * 1024 * 1024):
        p, v, grads = host_case(n, W, dtype, seed=chunk % 97, pinned=pinned)
        grads_in = list(grads)
        grads_in[3] = None
        p_np, v_np = p.numpy().copy(), v.numpy().copy()
        g_np = [None if g is None else grad_to_numpy(g) for g in grads_in]
        O.group_update_f32(p_np, v_np, g_np, off, mem, np.float32(0.1), 0.9, 1e-4)
        ws = torch.empty(B.star_host_workspace_bytes(5, dtype, chunk), dtype=torch.uint8, device="cuda")
        before = B.star_launch_count()
        B.star_group_update_host(p, v, grads_in, off, mem, 0.1, 0.9, 1e-4, ws)
        torch.cuda.current_stream().synchronize()
        want_chunks = min((n + chunk - 1) // chunk, (n + 2047) // 2048)
        assert B.star_launch_count() - before == want_chunks
        assert_matches(p, p_np, "params chunk=%d" % chunk)
        assert_matches(v, v_np, "momentum chunk=%d" % chunk)


def test_back_to_back_host_rounds_share_a_workspace(B):
    n, W = 300_000, 3
    p, v, grads = host_case(n, W, torch.bfloat16, seed=5, pinned=True)
    p_np, v_np = p.numpy().copy(), v.numpy().copy()
    g_np = [grad_to_numpy(g) for g in grads]
    ws = torch.empty(B.star_host_workspace_bytes(3, torch.bfloat16, 32768), dtype=torch.uint8, device="cuda")
    for off, mem in (([0, 3], [0, 1, 2]), ([0, 1, 2, 3], [2, 1, 0]), ([0, 2], [1, 2])):
        B.star_group_update_host(p, v, grads, off, mem, 0.05, 0.9, 0.01, ws)
        O.group_update_f32(p_np, v_np, g_np, off, mem, np.float32(0.05), 0.9, 0.01)
    torch.cuda.current_stream().synchronize()
    assert_matches(p, p_np, "params")
    assert_matches(v, v_np, "momentum")


def test_host_errors(B):
    p, v, grads = host_case(5000, 2, torch.bfloat16, seed=1, pinned=False)
    p0 = p.clone()
    tiny = torch.empty(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.StarError) as e:
        B.star_group_update_host(p, v, grads, [0, 2], [0, 1], 0.1, 0.9, 0.0, tiny)
    assert e.value.status == B.STAR_ERR_WORKSPACE_TOO_SMALL
    ws = torch.empty(B.star_host_workspace_bytes(2, torch.bfloat16, 2048), dtype=torch.uint8, device="cuda")
    with pytest.raises(B.StarError) as e:
        B.star_group_update_host(p, v, grads, [0, 0, 2], [0, 1], 0.1, 0.9, 0.0, ws)
    assert e.value.status == B.STAR_ERR_BAD_SCHEDULE
    with pytest.raises(B.StarError) as e:
        B.star_group_update_host(p, v, [grads[0], None], [0, 2], [0, 1], 0.1, 0.9, 0.0, ws)
    assert e.value.status == B.STAR_ERR_NULL_POINTER
    with pytest.raises(B.StarError):
        B.star_host_workspace_bytes(2, torch.bfloat16, 1000)
    torch.cuda.synchronize()
    assert torch.equal(p, p0)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("snap_dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("order", ["linear", "tree"])
def test_host_round_with_rates_snapshots_and_order(B, dtype, snap_dtype, order):
    """Per-group rates, snapshots into host tensors and the tree order through the
    chunked host path: the oracle's bits, snapshots included."""
    n, W = 300_007, 7
    off, mem = [0, 5, 6, 7], [6, 0, 4, 2, 5, 1, 3]            # a group of 5: tree and linear orders differ
    lrs = [0.1, 0.025, 0.05]
    for chunk in (2048, 65536):
        p, v, grads = host_case(n, W, dtype, seed=chunk % 89 + 3, pinned=True)
        snaps = [torch.zeros(n, dtype=snap_dtype).pin_memory(), None, torch.zeros(n, dtype=snap_dtype).pin_memory()]
        p_np, v_np = p.numpy().copy(), v.numpy().copy()
        snap_np = np.uint16 if snap_dtype == torch.bfloat16 else np.float32
        want = [np.zeros(n, snap_np), None, np.zeros(n, snap_np)]
        O.group_update_f32(p_np, v_np, [grad_to_numpy(g) for g in grads], off, mem, np.array(lrs, np.float32),
                           0.9, 1e-3, snapshots=want, sum_order=order)
        ws = torch.empty(B.star_host_workspace_bytes_ex(W, dtype, 2, snap_dtype, chunk), dtype=torch.uint8,
                         device="cuda")
        B.star_group_update_host_ex(p, v, grads, off, mem, lrs, 0.9, 1e-3, ws, snapshots=snaps,
                                    sum_order=B.STAR_SUM_TREE if order == "tree" else B.STAR_SUM_LINEAR)
        torch.cuda.current_stream().synchronize()
        assert_matches(p, p_np, "params chunk=%d" % chunk)
        assert_matches(v, v_np, "momentum chunk=%d" % chunk)
        for k in (0, 2):
            if snap_dtype == torch.bfloat16:
                assert np.array_equal(snaps[k].view(torch.int16).numpy().view(np.uint16), want[k]), "snapshot %d" % k
            else:
                assert_matches(snaps[k], want[k], "snapshot %d" % k)


def test_host_ex_errors(B):
    p, v, grads = host_case(5000, 2, torch.bfloat16, seed=2, pinned=False)
    p0 = p.clone()
    ws = torch.empty(B.star_host_workspace_bytes_ex(2, torch.bfloat16, 1, torch.float32, 2048), dtype=torch.uint8,
                     device="cuda")
    with pytest.raises(B.StarError) as e:                      # snapshot buffer is the parameter buffer
        B.star_group_update_host_ex(p, v, grads, [0, 2], [0, 1], [0.1], 0.9, 0.0, ws, snapshots=[p])
    assert e.value.status == B.STAR_ERR_INVALID_ARG
    s = torch.zeros(5000)
    with pytest.raises(B.StarError) as e:                      # two groups into one buffer
        B.star_group_update_host_ex(p, v, grads, [0, 1, 2], [0, 1], [0.1, 0.1], 0.9, 0.0, ws, snapshots=[s, s])
    assert e.value.status == B.STAR_ERR_INVALID_ARG
    with pytest.raises(B.StarError) as e:                      # two snapshots do not fit a workspace sized for one
        B.star_group_update_host_ex(p, v, grads, [0, 1, 2], [0, 1], [0.1, 0.1], 0.9, 0.0, ws,
                                    snapshots=[s, torch.zeros(5000)])
    assert e.value.status == B.STAR_ERR_WORKSPACE_TOO_SMALL
    torch.cuda.synchronize()
    assert torch.equal(p, p0)
