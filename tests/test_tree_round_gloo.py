"""The round over a communication tree as a protocol between ranks, on CPU.

Seven gloo ranks: six workers and the root (the parameter server).  The library
builds the tree from per-round latencies (Section IV-D2b: slower workers lower);
``TreeRound`` moves the partial sums up and the parameters down.  The arithmetic
steps are injected (the CPU oracle's functions here, the library's kernels on
GPU ranks), so the test checks the protocol: who forwards what to whom and in
which order the buffers are added.  Every rank must end with exactly the bits of
the single-process tree oracle (``oracle/tree_round.py``)."""
import os

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import tree_round as TR
from paper_2512_09685_b200 import binding as B
from paper_2512_09685_b200.tree_round import TreePlan, TreeRound
from tests.test_all_reduce_gloo import OracleBackend, _free_port, as_numpy

WORKERS = 6
N = 5_003
# latency per worker and fan-out per round: a two-level binary tree, a chain, a flat tree
ROUNDS = [([3.0, 1.0, 5.0, 2.0, 4.0, 6.0], 2), ([2.0, 1.0, 3.0, 6.0, 5.0, 4.0], 1), ([1.0] * 6, 6)]
LR, MU, WD = 0.05, 0.9, 1e-4


def inputs(dtype, round_index):
    g = torch.Generator().manual_seed(500 + round_index)
    return [(torch.randn(N, generator=g) * 0.01).to(dtype) for _ in range(WORKERS)]


def initial_state():
    g = torch.Generator().manual_seed(3)
    return torch.randn(N, generator=g) * 0.05, torch.randn(N, generator=g) * 0.02


def _rank_main(rank, port, dtype_name, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=WORKERS + 1)
    try:
        dtype = getattr(torch, dtype_name)
        p, v = initial_state()
        if rank < WORKERS:
            p = torch.zeros(N)                       # workers learn the parameters from the root
        runner = TreeRound(dist, rank, WORKERS + 1, backend=OracleBackend())
        for r, (latency, fanout) in enumerate(ROUNDS):
            parent_of = B.star_build_tree(latency, fanout)
            grad = inputs(dtype, r)[rank] if rank < WORKERS else None
            runner.run(grad, p, v if rank == WORKERS else None, parent_of, LR, MU, WD)
            np.save(os.path.join(out_dir, "p_%d_%d.npy" % (r, rank)), p.numpy())
            if rank == WORKERS:
                np.save(os.path.join(out_dir, "v_%d.npy" % r), v.numpy())
        dist.barrier()
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("dtype_name", ["float32", "bfloat16"])
def test_six_workers_and_a_root_reproduce_the_tree_oracle(tmp_path, dtype_name):
    mp.spawn(_rank_main, args=(_free_port(), dtype_name, str(tmp_path)), nprocs=WORKERS + 1, join=True)
    dtype = getattr(torch, dtype_name)
    p0, v0 = initial_state()
    p, v = p0.numpy().copy(), v0.numpy().copy()
    depths = []
    for r, (latency, fanout) in enumerate(ROUNDS):
        parent_of = TR.build_tree(latency, fanout)
        TR.tree_round_f32(p, v, [as_numpy(g) for g in inputs(dtype, r)], parent_of, LR, MU, WD)
        for rank in range(WORKERS + 1):
            got = np.load(tmp_path / ("p_%d_%d.npy" % (r, rank)))
            assert np.array_equal(got.view(np.uint32), p.view(np.uint32)), "round %d rank %d params" % (r, rank)
        got = np.load(tmp_path / ("v_%d.npy" % r))
        assert np.array_equal(got.view(np.uint32), v.view(np.uint32)), "round %d momentum" % r
        plan = TreePlan(parent_of)
        depth = lambda w: 0 if parent_of[w] < 0 else 1 + depth(parent_of[w])        # noqa: E731
        depths.append(max(depth(w) for w in range(WORKERS)))
        assert len(plan.top) == min(fanout, WORKERS)
    assert depths == [1, 5, 0]                       # two levels, a chain, a flat tree


def test_tree_plan_rejects_what_is_not_a_tree():
    TreePlan([-1, 0, 0, 1])
    for bad in ([1, 0], [0], [-1, 5], [-2, -1]):
        with pytest.raises(ValueError):
            TreePlan(bad)
