"""Multi-rank host logic on CPU: two gloo ranks shard a batch with no data-path collective, and
the benchmark's max-over-ranks reduction works."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import shard_oracle
from paper_2608_07524_b200 import binding as B
from paper_2608_07524_b200 import inputs
from paper_2608_07524_b200.shard import imbalance, shard_sequences


def test_shard_oracle_pins():
    # hand-worked: lengths 5, 4, 3, 3, 2 on two ranks -> work 25, 16, 9, 9, 4.
    # 25 -> rank 0 (25, 0); 16 -> rank 1 (25, 16); 9 -> rank 1 (25, 25); 9 -> rank 0, the lower rank of a tie
    # (34, 25); 4 -> rank 1 (34, 29)
    assert shard_oracle.shard_lpt([5, 4, 3, 3, 2], 2) == ([0, 1, 1, 0, 1], [34, 29])
    # input order does not matter for who gets what work; ties go to the lower index first
    assert shard_oracle.shard_lpt([3, 2, 5, 3, 4], 2) == ([1, 1, 0, 0, 1], [34, 29])
    # Graham's bound for longest-first greedy against the exhaustive optimum
    rng = np.random.default_rng(3)
    for _ in range(150):
        n, m = int(rng.integers(1, 9)), int(rng.integers(1, 5))
        lengths = [int(x) for x in rng.integers(1, 60, size=n)]
        rank_of, load = shard_oracle.shard_lpt(lengths, m)
        assert len(rank_of) == n and all(0 <= r < m for r in rank_of)
        assert load == [sum(L * L for L, r in zip(lengths, rank_of) if r == k) for k in range(m)]
        opt = shard_oracle.best_makespan(lengths, m)
        assert opt <= max(load) and 3 * m * max(load) <= (4 * m - 1) * opt


def test_library_sharding_matches_the_oracle():
    rng = np.random.default_rng(4)
    for _ in range(500):
        n, m = int(rng.integers(0, 40)), int(rng.integers(1, 9))
        lengths = [int(x) for x in rng.choice([0, 1, 7, 7, 100, 100, 4096, 46800, 131072], size=n)]
        assert B.dcp_shard_sequences(lengths, m) == shard_oracle.shard_lpt(lengths, m)
    assert B.dcp_shard_sequences([46341, 46341, 1], 1)[1] == [2 * 46341 ** 2 + 1]      # beyond 32 bits


def test_shards_partition_and_balance():
    lengths = inputs.video_lengths()
    for world in (1, 2, 4, 8):
        owned = shard_sequences(lengths, world)
        assert sorted(i for idx in owned for i in idx) == list(range(len(lengths)))
    # one 46800-token sequence dominates sum L^2, so two ranks cannot balance; the longest still
    # sits alone with the short ones elsewhere
    owned = shard_sequences(lengths, 2)
    longest = lengths.index(max(lengths))
    r = next(r for r in range(2) if longest in owned[r])
    assert owned[r] == [longest]
    assert imbalance(inputs.text_lengths(), 2) < 1.05


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    lengths = inputs.text_lengths()
    mine = shard_sequences(lengths, world)[rank]
    gathered = [None] * world
    dist.all_gather_object(gathered, mine)
    t = torch.tensor([10.0 + rank])                      # stand-in for this rank's elapsed time
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    tokens = torch.tensor([float(sum(lengths[i] for i in mine))])
    dist.all_reduce(tokens, op=dist.ReduceOp.SUM)
    if rank == 0:
        out.put((gathered, float(t), float(tokens)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    gathered, tmax, tokens = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    lengths = inputs.text_lengths()
    assert sorted(gathered[0] + gathered[1]) == list(range(len(lengths)))
    assert tmax == 11.0 and tokens == float(sum(lengths))
