"""Every element of the two largest flat workloads, at full size and over all
their rounds, against the oracle (run on all host cores over disjoint index
ranges: the path is elementwise, so the split changes nothing)."""
import threading

import numpy as np
import psutil
import pytest
import torch

from oracle import star_oracle as O
from paper_2512_09685_b200 import workloads as WL
from tests.parity import grad_to_numpy

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["cfg2_bert_large", "cfg3_vgg16_asgd"])
def test_every_element_of_every_round(name):
    from paper_2512_09685_b200 import binding as B
    w = WL.BY_NAME[name]
    n = w.n
    need = n * (w.W * w.grad_bytes + 24)
    if psutil.virtual_memory().available < 2 * need:
        pytest.skip("needs %.0f GB of free host memory" % (2 * need / 1e9))
    p = WL.make_params(w, "cuda")[0]
    v = WL.make_momentum(w, "cuda")[0]
    p_np, v_np = p.cpu().numpy().copy(), v.cpu().numpy().copy()
    grads = [torch.empty(n, dtype=w.torch_grad_dtype(), device="cuda") for _ in range(w.W)]
    threads = max(1, min(16, len(psutil.Process().cpu_affinity())))
    bounds = [n * i // threads for i in range(threads + 1)]
    for step in range(w.steps):
        for wk in range(w.W):
            WL.fill_grads(w, step, wk, [grads[wk]])
        off, mem = B.encode(w.decision(step))
        B.star_group_update(p, v, grads, off, mem, w.lr, w.mu, w.wd)
        g_np = [grad_to_numpy(g) for g in grads]

        def work(i):
            a, b = bounds[i], bounds[i + 1]
            O.group_update_f32(p_np[a:b], v_np[a:b], [g[a:b] for g in g_np], off, mem, np.float32(w.lr),
                               w.mu, w.wd)
        pool = [threading.Thread(target=work, args=(i,)) for i in range(threads)]
        for t in pool:
            t.start()
        for t in pool:
            t.join()
        torch.cuda.synchronize()
        for got, want, what in ((p, p_np, "params"), (v, v_np, "momentum")):
            got = got.cpu().numpy()
            differ = int((got.view(np.uint32) != want.view(np.uint32)).sum())
            assert differ == 0, "%s step %d: %d of %d %s elements differ" % (name, step, differ, n, what)


def test_every_element_of_the_tensor_list_in_every_round():
    """The 292-tensor GPT-2-medium list through the one-launch tensor-list kernel,
    all 354,823,168 elements after each of the 5 rounds (2..8 groups per round)."""
    from paper_2512_09685_b200 import binding as B
    w = WL.BY_NAME["cfg4_gpt2_medium"]
    n, sizes = w.n, w.sizes
    need = n * (w.W * w.grad_bytes + 24)
    if psutil.virtual_memory().available < 2 * need:
        pytest.skip("needs %.0f GB of free host memory" % (2 * need / 1e9))
    params = WL.make_params(w, "cuda")
    momentum = WL.make_momentum(w, "cuda")
    p_np = torch.cat(params).cpu().numpy().copy()
    v_np = torch.cat(momentum).cpu().numpy().copy()
    grads = [[torch.empty(s, dtype=torch.bfloat16, device="cuda") for s in sizes] for _ in range(w.W)]
    ws = torch.empty(B.star_multi_workspace_bytes(sizes, w.W), dtype=torch.uint8, device="cuda")
    plan = B.star_multi_prepare(params, momentum, grads, ws)
    threads = max(1, min(16, len(psutil.Process().cpu_affinity())))
    bounds = [n * i // threads for i in range(threads + 1)]
    for step in range(w.steps):
        for wk in range(w.W):
            WL.fill_grads(w, step, wk, grads[wk])
        off, mem = B.encode(w.decision(step))
        before = B.star_launch_count()
        B.star_group_update_multi(plan, off, mem, w.lr, w.mu, w.wd)
        assert B.star_launch_count() == before + 1
        g_np = [grad_to_numpy(torch.cat(grads[wk])) for wk in range(w.W)]

        def work(i):
            a, b = bounds[i], bounds[i + 1]
            O.group_update_f32(p_np[a:b], v_np[a:b], [g[a:b] for g in g_np], off, mem, np.float32(w.lr),
                               w.mu, w.wd)
        pool = [threading.Thread(target=work, args=(i,)) for i in range(threads)]
        for t in pool:
            t.start()
        for t in pool:
            t.join()
        torch.cuda.synchronize()
        for got, want, what in ((params, p_np, "params"), (momentum, v_np, "momentum")):
            got = torch.cat(got).cpu().numpy()
            differ = int((got.view(np.uint32) != want.view(np.uint32)).sum())
            assert differ == 0, "step %d (%d groups): %d of %d %s elements differ" % (
                step, len(off) - 1, differ, n, what)
