"""The N > 1 path is token-parallel replicas with no data-path collective; its host-side logic (which tokens /
batches a rank owns, barrier + max-over-ranks timing, aggregate throughput) is covered here with two gloo
ranks on CPU.  The per-rank result is the oracle's, so the union over ranks must equal the single-rank result."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2603_15965_b200 import shard
from paper_2603_15965_b200 import workloads as W


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = W.random_problem(77, 203, 4, 32, 48, 8, "f32", unrouted_frac=0.1)
        p = w.projections[0]
        lo, hi = shard.token_range(w.N, rank, world)
        # every rank runs the whole path on its own tokens only: nothing is exchanged
        r = w.r[lo:hi]
        counts, offsets, perm = oracle.group(r, w.C)
        h, products = oracle.apply(w.inputs["x"][lo:hi], p.y[lo:hi], p.A, p.B, r)
        np.save(os.path.join(out_dir, f"h{rank}.npy"), h)
        dist.barrier()
        # timing bookkeeping: the slowest rank defines the step
        ms = shard.max_over_ranks(1.0 + rank, dist)
        assert ms == float(world)
        total = torch.tensor([products], dtype=torch.int64)
        dist.all_reduce(total)
        assert int(total.item()) == int(np.count_nonzero(w.r >= 0))
        assert shard.rank_batches(rank, world, 3) == [rank * 3, rank * 3 + 1, rank * 3 + 2]
    finally:
        dist.destroy_process_group()


def test_two_rank_token_sharding_matches_single_rank(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    w = W.random_problem(77, 203, 4, 32, 48, 8, "f32", unrouted_frac=0.1)
    p = w.projections[0]
    ref, _ = oracle.apply(w.inputs["x"], p.y, p.A, p.B, w.r)
    got = np.concatenate([np.load(tmp_path / f"h{r}.npy") for r in range(world)])
    assert np.array_equal(got, ref)                      # rows are independent: sharding changes nothing, bit for bit


def test_token_ranges_partition_the_batch():
    for n, world in [(0, 3), (5, 8), (4096, 2), (4097, 4), (16384, 8)]:
        ranges = [shard.token_range(n, r, world) for r in range(world)]
        assert ranges[0][0] == 0 and ranges[-1][1] == n
        assert all(a[1] == b[0] for a, b in zip(ranges, ranges[1:]))
        sizes = [hi - lo for lo, hi in ranges]
        assert max(sizes) - min(sizes) <= 1
    assert shard.aggregate_tokens_per_s(4096, 2, 0.05) == 2 * 4096 / 5e-5
    assert shard.max_over_ranks(3.5) == 3.5
