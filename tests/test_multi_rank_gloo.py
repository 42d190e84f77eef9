"""The multi-rank host logic on CPU: two gloo ranks own disjoint shards of one
tensor (library shard helper), run the round on their shard with no exchange,
and together reproduce the single-process result; the benchmark's time
reduction reports the slowest rank."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import star_oracle as O
from paper_2512_09685_b200 import binding as B
from paper_2512_09685_b200 import workloads as WL


def test_shard_ranges_partition_the_index_space():
    for n in (0, 1, 15, 16, 17, 1000, 25_557_032):
        for world in (1, 2, 3, 8):
            for align in (1, 16):
                pos, counts = 0, []
                for rank in range(world):
                    first, count = B.star_shard_range(n, world, rank, align)
                    assert first == pos and first % align == 0 or count == 0
                    pos = first + count
                    counts.append(count)
                assert pos == n and sum(counts) == n
                assert max(counts) - min(counts) < 2 * align
    with pytest.raises(B.StarError):
        B.star_shard_range(10, 2, 2, 16)
    with pytest.raises(B.StarError):
        B.star_shard_range(10, 0, 0, 16)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, n, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import bench
        w = WL.scaled(WL.BY_NAME["cfg1_resnet50"], n)
        # every rank generates the same seeded tensors and keeps only its shard
        first, count = B.star_shard_range(n, world, rank, 16)
        p = WL.make_params(w, "cpu")[0][first:first + count].numpy().copy()
        v = np.zeros(count, np.float32)
        grads = [g[0][first:first + count].view(torch.int16).numpy().view(np.uint16).copy()
                 for g in WL.make_grads(w, 0, "cpu")]
        off, mem = B.encode(w.decision(0))
        O.group_update_f32(p, v, grads, off, mem, np.float32(w.lr), w.mu, w.wd)   # no exchange
        # gather only to CHECK the result (not part of the path)
        sizes = [B.star_shard_range(n, world, r, 16)[1] for r in range(world)]
        padded = torch.zeros(max(sizes))
        padded[:count] = torch.from_numpy(p)
        parts = [torch.empty(max(sizes)) for _ in sizes]
        dist.all_gather(parts, padded)
        parts = [part[:s] for part, s in zip(parts, sizes)]
        slowest = bench.max_over_ranks(1.0 + rank, dist, "cpu")
        if rank == 0:
            np.save(os.path.join(out_dir, "p.npy"), torch.cat(parts).numpy())
            np.save(os.path.join(out_dir, "t.npy"), np.array([slowest]))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_reproduce_the_single_process_round(tmp_path):
    n, world = 100_003, 2
    mp.spawn(_rank_main, args=(world, _free_port(), n, str(tmp_path)), nprocs=world, join=True)
    got = np.load(tmp_path / "p.npy")
    w = WL.scaled(WL.BY_NAME["cfg1_resnet50"], n)
    p = WL.make_params(w, "cpu")[0].numpy().copy()
    v = np.zeros(n, np.float32)
    grads = [g[0].view(torch.int16).numpy().view(np.uint16).copy() for g in WL.make_grads(w, 0, "cpu")]
    off, mem = B.encode(w.decision(0))
    O.group_update_f32(p, v, grads, off, mem, np.float32(w.lr), w.mu, w.wd)
    assert np.array_equal(got.view(np.uint32), p.view(np.uint32))
    assert np.load(tmp_path / "t.npy")[0] == 2.0          # max over ranks of (1.0, 2.0)
