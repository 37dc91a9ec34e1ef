"""Multi-rank host logic on CPU (gloo, world size 2): batch sharding covers every sequence
exactly once, results gathered from the ranks equal the single-rank result, and the
whole-job rate uses the slowest rank's time.  The per-sequence work here is the oracle's
walk, which stands in for the GPU call; the CUDA path is not involved."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2502_06352_b200.shard import shard_range, whole_job_rate


def test_shard_range_partitions():
    for total in (0, 1, 7, 8, 64, 65):
        for world in (1, 2, 3, 8):
            got = []
            for r in range(world):
                b, e = shard_range(total, r, world)
                assert 0 <= b <= e <= total and e - b in (total // world, total // world + 1)
                got += list(range(b, e))
            assert got == list(range(total))
    assert whole_job_rate([100, 100], 50.0) == 4000.0


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    B, N = 7, 5
    rng = np.random.default_rng(0)                  # the same job description on every rank
    nxt = rng.integers(-1, 2, (B, N))
    b, e = shard_range(B, rank, world)
    # per-sequence result: number of accepted hops from node 0 following nxt (a chain walk)
    local = torch.full((B,), -1, dtype=torch.int64)
    for s in range(b, e):
        cur, hops = 0, 0
        while nxt[s, cur] > 0 and cur + nxt[s, cur] < N:
            cur += int(nxt[s, cur])
            hops += 1
        local[s] = hops
    # owners hold their entries, others -1: MAX over ranks assembles the batch
    dist.all_reduce(local, op=dist.ReduceOp.MAX)
    t = torch.tensor([10.0 + 5.0 * rank], dtype=torch.float64)      # pretend device time, ms
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    units = torch.tensor([float(e - b)], dtype=torch.float64)
    dist.all_reduce(units, op=dist.ReduceOp.SUM)
    if rank == 0:
        torch.save(dict(result=local, t=float(t), units=float(units)), out)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_assemble_the_single_rank_result(tmp_path):
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    out = str(tmp_path / "r0.pt")
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    got = torch.load(out)
    # single-rank reference
    B, N = 7, 5
    nxt = np.random.default_rng(0).integers(-1, 2, (B, N))
    want = []
    for s_ in range(B):
        cur, hops = 0, 0
        while nxt[s_, cur] > 0 and cur + nxt[s_, cur] < N:
            cur += int(nxt[s_, cur])
            hops += 1
        want.append(hops)
    assert got["result"].tolist() == want
    assert got["t"] == 15.0 and got["units"] == 7.0
    assert whole_job_rate([4, 3], got["t"]) == 7 / 0.015
