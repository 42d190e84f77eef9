"""GPU parity on the five workloads at their full sizes, in the launch
configuration the benchmark times.  The oracle follows a sample of the elements
(all of them where that takes seconds): the path is elementwise, so the oracle
run on gathered elements is exactly the oracle on those elements."""
import numpy as np
import pytest
import torch

from oracle import schedule as S
from oracle import star_oracle as O
from paper_2512_09685_b200 import workloads as WL
from tests.parity import assert_matches, grad_to_numpy, sample_indices

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2512_09685_b200 import binding
    return binding


def oracle_schedule(decision):
    if decision.kind == "labels":
        return S.from_labels(decision.labels)
    if decision.kind == "static_x":
        return S.static_x(decision.arrival_order, decision.W, decision.x, decision.sort_members)
    return S.dynamic_x(decision.iter_time, decision.labels)


def run_flat(B, w, full_oracle):
    dev = "cuda"
    p = WL.make_params(w, dev)[0]
    v = WL.make_momentum(w, dev)[0]
    n = w.n
    idx_np = np.arange(n, dtype=np.int64) if full_oracle else sample_indices(n, w.seed)
    idx = torch.from_numpy(idx_np).to(dev)
    p_ref = p[idx].cpu().numpy().copy()
    v_ref = v[idx].cpu().numpy().copy()
    p_before = p.clone()
    grads = [torch.empty(n, dtype=w.torch_grad_dtype(), device=dev) for _ in range(w.W)]
    for step in range(w.steps):
        for wk in range(w.W):
            WL.fill_grads(w, step, wk, [grads[wk]])
        decision = w.decision(step)
        off, mem = B.encode(decision)
        assert (off, mem) == tuple(oracle_schedule(decision))
        B.star_group_update(p, v, grads, off, mem, w.lr, w.mu, w.wd)
        g_np = [grad_to_numpy(g[idx]) for g in grads]
        O.group_update_f32(p_ref, v_ref, g_np, off, mem, np.float32(w.lr), w.mu, w.wd)
        torch.cuda.synchronize()
        assert_matches(p[idx], p_ref, "%s step %d params" % (w.name, step))
        assert_matches(v[idx], v_ref, "%s step %d momentum" % (w.name, step))
    # properties over the whole arrays: finite, and every element was updated
    assert bool(torch.isfinite(p).all()) and bool(torch.isfinite(v).all())
    assert (p != p_before).float().mean().item() > 0.999
    assert (v != 0).float().mean().item() > 0.999


def test_cfg0_small_fp32_full(B):
    run_flat(B, WL.BY_NAME["cfg0_small_f32"], full_oracle=True)


def test_cfg1_resnet50_sized_full(B):
    run_flat(B, WL.BY_NAME["cfg1_resnet50"], full_oracle=True)


def test_cfg2_bert_large_sized_sampled(B):
    run_flat(B, WL.BY_NAME["cfg2_bert_large"], full_oracle=False)


def test_cfg3_vgg16_sized_asgd_sampled(B):
    run_flat(B, WL.BY_NAME["cfg3_vgg16_asgd"], full_oracle=False)


def test_cfg4_gpt2_medium_tensor_list_sampled(B):
    w = WL.BY_NAME["cfg4_gpt2_medium"]
    dev = "cuda"
    params = WL.make_params(w, dev)
    momentum = WL.make_momentum(w, dev)
    sizes = w.sizes
    assert len(params) == 292
    grads = [[torch.empty(s, dtype=torch.bfloat16, device=dev) for s in sizes] for _ in range(w.W)]
    ws = torch.empty(B.star_multi_workspace_bytes(sizes, w.W), dtype=torch.uint8, device=dev)
    plan = B.star_multi_prepare(params, momentum, grads, ws)
    assert plan.total_elements == w.n == 354_823_168
    # sample: small tensors whole, big ones head / tail / random runs
    idx = [torch.from_numpy(sample_indices(s, 1000 + t, chunk=2048, n_chunks=6)).to(dev)
           for t, s in enumerate(sizes)]
    gather = lambda tensors: torch.cat([x[i] for x, i in zip(tensors, idx)])
    p_ref = gather(params).cpu().numpy().copy()
    v_ref = gather(momentum).cpu().numpy().copy()
    ks = set()
    for step in range(w.steps):
        for wk in range(w.W):
            WL.fill_grads(w, step, wk, grads[wk])
        decision = w.decision(step)
        off, mem = B.encode(decision)
        assert (off, mem) == tuple(oracle_schedule(decision))
        ks.add(len(off) - 1)
        before = B.star_launch_count()
        B.star_group_update_multi(plan, off, mem, w.lr, w.mu, w.wd)
        assert B.star_launch_count() - before == 1            # one launch for 292 tensors
        g_np = [grad_to_numpy(gather(grads[wk])) for wk in range(w.W)]
        O.group_update_f32(p_ref, v_ref, g_np, off, mem, np.float32(w.lr), w.mu, w.wd)
        torch.cuda.synchronize()
        assert_matches(gather(params), p_ref, "gpt2 step %d params" % step)
        assert_matches(gather(momentum), v_ref, "gpt2 step %d momentum" % step)
    assert all(bool(torch.isfinite(p).all()) for p in params)
    assert all(bool((v != 0).float().mean() > 0.99) for v in momentum)
    assert len(ks) >= 2


@pytest.mark.parametrize("mode", ["snap_f32", "snap_bf16", "tree"])
def test_cfg1_extended_entry_point_every_element(B, mode):
    """The ResNet-50-sized workload through star_group_update_ex as the benchmark
    times it (one snapshot per group, or tree order): every element of p, v and
    of every snapshot, two rounds."""
    w = WL.BY_NAME["cfg1_resnet50"]
    n = w.n
    p = WL.make_params(w, "cuda")[0]
    v = WL.make_momentum(w, "cuda")[0]
    p_np, v_np = p.cpu().numpy().copy(), v.cpu().numpy().copy()
    grads = [torch.empty(n, dtype=torch.bfloat16, device="cuda") for _ in range(w.W)]
    snap_dtype = {"snap_f32": torch.float32, "snap_bf16": torch.bfloat16}.get(mode)
    for step in range(2):
        for wk in range(w.W):
            WL.fill_grads(w, step, wk, [grads[wk]])
        off, mem = B.encode(w.decision(step))
        K = len(off) - 1
        lrs = [w.lr * (k + 1) / K for k in range(K)]              # distinct rates per group
        snaps = [torch.empty(n, dtype=snap_dtype, device="cuda") for _ in range(K)] if snap_dtype else None
        B.star_group_update_ex(p, v, grads, off, mem, lrs, w.mu, w.wd, snapshots=snaps,
                               sum_order=B.STAR_SUM_TREE if mode == "tree" else B.STAR_SUM_LINEAR)
        want = None
        if snap_dtype:
            want = [np.zeros(n, np.uint16 if snap_dtype == torch.bfloat16 else np.float32) for _ in range(K)]
        O.group_update_f32(p_np, v_np, [grad_to_numpy(g) for g in grads], off, mem, np.array(lrs, np.float32),
                           w.mu, w.wd, snapshots=want, sum_order="tree" if mode == "tree" else "linear")
        torch.cuda.synchronize()
        assert_matches(p, p_np, "%s step %d params" % (mode, step))
        assert_matches(v, v_np, "%s step %d momentum" % (mode, step))
        for k in range(K if snap_dtype else 0):
            if snap_dtype == torch.bfloat16:
                got = snaps[k].cpu().view(torch.int16).numpy().view(np.uint16)
                assert np.array_equal(got, want[k]), "%s step %d snapshot %d" % (mode, step, k)
            else:
                assert_matches(snaps[k], want[k], "%s step %d snapshot %d" % (mode, step, k))


def test_cfg4_list_with_snapshot_sets_sampled(B):
    """The GPT-2-medium list through star_group_update_multi_ex as the benchmark
    times it (per-group rates, one bf16 snapshot set per group): sampled elements
    of p, v and of every written snapshot set, two rounds."""
    w = WL.BY_NAME["cfg4_gpt2_medium"]
    sizes, dev = w.sizes, "cuda"
    params = WL.make_params(w, dev)
    momentum = WL.make_momentum(w, dev)
    grads = [[torch.empty(s, dtype=torch.bfloat16, device=dev) for s in sizes] for _ in range(w.W)]
    sets = [[torch.zeros(s, dtype=torch.bfloat16, device=dev) for s in sizes] for _ in range(8)]
    ws = torch.empty(B.star_multi_workspace_bytes_ex(sizes, w.W, 8), dtype=torch.uint8, device=dev)
    plan = B.star_multi_prepare_ex(params, momentum, grads, sets, ws)
    idx = [torch.from_numpy(sample_indices(s, 2000 + t, chunk=2048, n_chunks=4)).to(dev) for t, s in enumerate(sizes)]
    gather = lambda tensors: torch.cat([x[i] for x, i in zip(tensors, idx)])
    p_ref, v_ref = gather(params).cpu().numpy().copy(), gather(momentum).cpu().numpy().copy()
    for step in range(2):
        for wk in range(w.W):
            WL.fill_grads(w, step, wk, grads[wk])
        off, mem = B.encode(w.decision(step))
        K = len(off) - 1
        lrs = [w.lr * (1 + k) for k in range(K)]
        choice = [(k * 3) % 8 for k in range(K)]                  # distinct sets, not in order
        before = B.star_launch_count()
        B.star_group_update_multi_ex(plan, off, mem, lrs, w.mu, w.wd, choice, B.STAR_SUM_LINEAR)
        assert B.star_launch_count() == before + 1
        want = [np.zeros(p_ref.size, np.uint16) for _ in range(K)]
        O.group_update_f32(p_ref, v_ref, [grad_to_numpy(gather(grads[wk])) for wk in range(w.W)], off, mem,
                           np.array(lrs, np.float32), w.mu, w.wd, snapshots=want)
        torch.cuda.synchronize()
        assert_matches(gather(params), p_ref, "step %d params" % step)
        assert_matches(gather(momentum), v_ref, "step %d momentum" % step)
        for k in range(K):
            got = gather(sets[choice[k]]).cpu().view(torch.int16).numpy().view(np.uint16)
            assert np.array_equal(got, want[k]), "step %d snapshot of group %d" % (step, k)
