"""The all-reduce architecture's round as a protocol between ranks, on CPU.

Five gloo ranks, one per worker.  The library's mode decision (Section II
straggler rule, Eq. 3) says which workers leave the ring and which of them
report in time; ``AllReduceRound`` moves the buffers (children -> parent, the
ring's exchange in either form, parent -> children).  The two arithmetic steps
are injected: on a GPU they are the library's kernels, here -- no GPU -- the
test hands in the CPU oracle's functions, so what is checked is the protocol:
who sends what to whom, in which order the buffers are summed, the report
count.  Every rank must end with exactly the bits of the single-process round
oracle (``oracle/all_reduce.py``)."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import all_reduce as AR
from oracle import star_oracle as O
from paper_2512_09685_b200 import binding as B
from paper_2512_09685_b200.all_reduce_round import AllReduceRound, RoundPlan

WORLD = 5
N = 10_007
# (iteration time in the ring, iteration time as a child, phi, t_w_max) per round.
# Round 0: workers 4 and 3 are stragglers; as children 4 is quick, 3 needs longer than any wait allowed.
# Round 1: only worker 1 is a straggler and it reports in time.  Round 2: nobody is removed.
ROUNDS = [
    ([1.0, 1.05, 0.95, 3.0, 5.0], [9.0, 9.0, 9.0, 2.5, 1.1], 1e4, 0.5),
    ([1.0, 4.0, 1.0, 1.1, 0.9], [9.0, 1.2, 9.0, 9.0, 9.0], 1e4, 0.5),
    ([1.0, 1.0, 1.1, 1.0, 1.05], [9.0] * 5, 10.0, 0.5),
]
LR, MU, WD, M = 0.05, 0.9, 1e-4, 128.0


def as_numpy(t: torch.Tensor) -> np.ndarray:
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


class OracleBackend:
    """The arithmetic steps on CPU tensors through the oracle (test only)."""

    def empty(self, n, dtype, like):
        return torch.empty(n, dtype=dtype)

    def reduce(self, out, buffers):
        out.copy_(torch.from_numpy(O.group_reduce_f32([as_numpy(b) for b in buffers], list(range(len(buffers))))))

    def update_from_sums(self, params, momentum, sums, n_reports, lr, mu, wd):
        p, v = params.numpy(), momentum.numpy()                   # views: updated in place
        O.update_from_sums_f32(p, v, [s.contiguous().numpy() for s in sums], n_reports, lr, mu, wd)


def inputs(dtype, round_index):
    """The same seeded tensors on every rank and in the checking process."""
    g = torch.Generator().manual_seed(1000 + round_index)
    grads = [(torch.randn(N, generator=g) * 0.01).to(dtype) for _ in range(WORLD)]
    return grads


def initial_state():
    g = torch.Generator().manual_seed(7)
    return torch.randn(N, generator=g) * 0.05, torch.randn(N, generator=g) * 0.02


def decide(round_index):
    t, child, phi, t_w_max = ROUNDS[round_index]
    x, t_w, T, removed, (off, mem) = B.star_choose_all_reduce_mode(t, child, phi, M, t_w_max)
    in_time = [w for w in mem if w in removed]
    return removed, in_time


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, port, dtype_name, exchange, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=WORLD)
    try:
        dtype = getattr(torch, dtype_name)
        p, v = initial_state()
        runner = AllReduceRound(dist, rank, WORLD, backend=OracleBackend(), exchange=exchange)
        for r in range(len(ROUNDS)):
            removed, in_time = decide(r)
            grad = inputs(dtype, r)[rank]
            runner.run(grad, p, v, removed, in_time, LR, MU, WD)
            np.save(os.path.join(out_dir, "p_%d_%d.npy" % (r, rank)), p.numpy())
            np.save(os.path.join(out_dir, "v_%d_%d.npy" % (r, rank)), v.numpy())
        dist.barrier()
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("dtype_name", ["float32", "bfloat16"])
@pytest.mark.parametrize("exchange", ["gather", "scatter"])
def test_five_ranks_reproduce_the_round_oracle(tmp_path, dtype_name, exchange):
    mp.spawn(_rank_main, args=(_free_port(), dtype_name, exchange, str(tmp_path)), nprocs=WORLD, join=True)
    dtype = getattr(torch, dtype_name)
    p0, v0 = initial_state()
    p, v = p0.numpy().copy(), v0.numpy().copy()
    seen = []
    for r in range(len(ROUNDS)):
        removed, in_time = decide(r)
        seen.append((len(removed), len(in_time)))
        ring = [w for w in range(WORLD) if w not in removed]
        parent_of = AR.assign_parents(removed, ring)
        grads = [as_numpy(g) for g in inputs(dtype, r)]
        AR.all_reduce_round_f32(p, v, grads, ring, parent_of, in_time, LR, MU, WD)
        for rank in range(WORLD):
            got = np.load(tmp_path / ("p_%d_%d.npy" % (r, rank)))
            assert np.array_equal(got.view(np.uint32), p.view(np.uint32)), "round %d rank %d params" % (r, rank)
            got = np.load(tmp_path / ("v_%d_%d.npy" % (r, rank)))       # children hold their parent's state
            assert np.array_equal(got.view(np.uint32), v.view(np.uint32)), "round %d rank %d momentum" % (r, rank)
    # the three rounds exercise: two removed with one late; one removed, in time; nobody removed
    assert seen == [(2, 1), (1, 1), (0, 0)]


def test_round_plan_counts_reports_as_eq3_does():
    plan = RoundPlan(9, removed=[8, 2, 5], in_time=[5, 8])
    assert plan.ring == [0, 1, 3, 4, 6, 7]
    assert plan.parent_of[8] == 0 and plan.parent_of[2] == 1 and plan.parent_of[5] == 3
    assert plan.children == {0: [8], 1: [], 3: [5], 4: [], 6: [], 7: []}
    assert plan.n_reports == 9 - 3 + 2
    with pytest.raises(ValueError):
        RoundPlan(4, removed=[3], in_time=[2])
