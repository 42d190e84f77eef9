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
