"""Edge cases at scale: a tensor with more than 2^31 elements (64-bit index
arithmetic), and stopping / reloading the state between rounds."""
import io
import json
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

from oracle import star_oracle as O
from tests.parity import assert_matches, grad_to_numpy

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_2512_09685_b200 import binding
    return binding


def test_more_than_two_to_the_31_elements(B):
    n = (1 << 31) + 4099                               # 8.6 GB each of p and v
    free, _ = torch.cuda.mem_get_info()
    if free < 40 * (1 << 30):
        pytest.skip("needs 40 GB of free device memory")
    g = torch.Generator(device="cuda").manual_seed(5)
    p = torch.empty(n, device="cuda")
    v = torch.empty(n, device="cuda")
    grads = [torch.empty(n, dtype=torch.bfloat16, device="cuda") for _ in range(3)]
    step = 1 << 28
    for t, std in [(p, 0.05), (v, 0.02)] + [(x, 0.01) for x in grads]:
        for a in range(0, n, step):
            b = min(n, a + step)
            t[a:b].copy_(torch.randn(b - a, generator=g, device="cuda") * std)
    # sample: head, tail, and runs around every point where a 32-bit element or
    # byte index would wrap (2^29, 2^30, 2^31 elements = 2^31, 2^32, 2^33 bytes of fp32)
    runs = [0, n - 5000] + [m - 2500 for m in (1 << 29, 1 << 30, 1 << 31, 3 << 29)]
    idx = torch.cat([torch.arange(a, a + 5000, device="cuda") for a in runs])
    p_np, v_np = p[idx].cpu().numpy().copy(), v[idx].cpu().numpy().copy()
    g_np = [grad_to_numpy(x[idx]) for x in grads]
    off, mem = [0, 2, 3], [2, 0, 1]
    for _ in range(2):
        B.star_group_update(p, v, grads, off, mem, 0.1, 0.9, 1e-4)
        O.group_update_f32(p_np, v_np, g_np, off, mem, np.float32(0.1), 0.9, 1e-4)
    torch.cuda.synchronize()
    assert_matches(p[idx], p_np, "params")
    assert_matches(v[idx], v_np, "momentum")
    for a in range(0, n, step):                        # every element was updated exactly like its neighbours
        assert bool(torch.isfinite(p[a:min(n, a + step)]).all())
    del p, v, grads
    torch.cuda.empty_cache()


def test_stop_reload_continue_equals_uninterrupted(B):
    """State = (p, v).  k rounds, serialize, reload into fresh buffers, m more
    rounds == k + m rounds without a break, bit for bit."""
    n, W = 300_007, 5
    g = torch.Generator(device="cuda").manual_seed(9)
    p0 = torch.randn(n, generator=g, device="cuda") * 0.05
    rounds = []
    for r in range(5):
        grads = [(torch.randn(n, generator=g, device="cuda") * 0.01).to(torch.bfloat16) for _ in range(W)]
        off, mem = B.star_schedule_static_x([(r + w) % W for w in range(W)], W, 1 + r % 3, True)
        rounds.append((grads, off, mem))
    p, v = p0.clone(), torch.zeros(n, device="cuda")
    for grads, off, mem in rounds:
        B.star_group_update(p, v, grads, off, mem, 0.05, 0.9, 1e-3)
    q, u = p0.clone(), torch.zeros(n, device="cuda")
    for grads, off, mem in rounds[:2]:
        B.star_group_update(q, u, grads, off, mem, 0.05, 0.9, 1e-3)
    blob = io.BytesIO()
    torch.save({"params": q.cpu(), "momentum": u.cpu(), "round": 2}, blob)
    del q, u
    blob.seek(0)
    state = torch.load(blob)
    q, u = state["params"].cuda(), state["momentum"].cuda()
    for grads, off, mem in rounds[state["round"]:]:
        B.star_group_update(q, u, grads, off, mem, 0.05, 0.9, 1e-3)
    torch.cuda.synchronize()
    assert torch.equal(p, q) and torch.equal(v, u)


def test_bench_line_on_a_small_case():
    """The benchmark's own JSON line (reduced size, device-timed part only)."""
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--steps", "5", "--warmup", "3",
                          "--n", "4000000", "--no-extra"], capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["unit"] == "GB/s" and d["n_gpus"] == 1 and d["steps"] == 5 and d["gpu_launches"] == 5
    assert d["value"] > 100 and d["scaling"] == "weak" and d["dtype"] == "f32" and d["data"] == "synthetic"
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["peak"] > 1000
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    assert r["traffic"] is None                        # reduced size: no capture applies
    assert set(d["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}
    regions = d["timed_regions"]
    assert regions["count"] >= 3 and regions["steps_each"] == 5
    assert regions["value_min"] <= d["value"] <= regions["value_max"]
    assert d["config"]["workload"] == "cfg4_gpt2_medium" and d["roofline"]["kernel"] == "star_update_multi_kernel"
    import bench
    from paper_2512_09685_b200 import workloads as WL
    reduced = WL.reduced_list(WL.BY_NAME["cfg4_gpt2_medium"], 2, 4000000 // 1024)
    assert d["config"] == bench.config_for(reduced, 1)            # the dict the reference arm prints for the same workload


def test_all_reduce_architecture_round_on_one_gpu():
    """One rank: a ring of one, nobody removed -- the aggregate and update
    kernels of the round still run (two launches per step)."""
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--architecture", "all_reduce",
                          "--steps", "5", "--warmup", "3", "--n", "4000000"], capture_output=True, text=True,
                         timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    d = json.loads([l for l in out.stdout.splitlines() if l.strip()][-1])
    assert d["config"]["architecture"] == "all_reduce" and d["n_gpus"] == 1
    assert d["gpu_launches"] == 10 and d["value"] > 100


def test_single_entry_runs_used_for_profiler_captures():
    """`--only NAME --n N`: one entry of other_workloads at a reduced size (the
    commands the profile summaries were captured with)."""
    for name, kernel in (("group_reduce_2_bf16_to_f32_100M", "star_group_reduce_kernel"),
                         ("tree_1x16_100M", "star_update_flat_snapshot_kernel"),
                         ("cfg4_gpt2_medium/snap_bf16", "star_update_multi_ex_kernel")):
        out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--n", "2000000", "--only", name],
                             capture_output=True, text=True, timeout=600, cwd=ROOT)
        assert out.returncode == 0, out.stderr[-2000:]
        d = json.loads([l for l in out.stdout.splitlines() if l.strip()][-1])["other_workloads"]
        assert list(d) == [name] and d[name]["roofline"]["kernel"] == kernel and d[name]["gbs"] > 50
