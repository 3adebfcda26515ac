"""World-size-2 CPU (gloo) check of the multi-GPU plumbing: per-rank workloads and job-level reduction."""
import os
import socket

import numpy as np
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2405_06219_b200 import sharding, workloads


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = sharding.rank_workload(workloads.configs()[1].scaled(context=64, batch=2), rank, world)
    tokens = float(w.lengths().sum())
    t, u = sharding.reduce_job(10.0 + rank, tokens)
    first = w.tokens("k", 0, 0, 4).astype(np.float32).sum()
    passes = sharding.reduce_max_list([1.0 + rank, 5.0 - rank, 2.0])      # per-pass timings: the slowest rank each
    est = sharding.reduce_max(3.0 * (rank + 1))
    job = sharding.reduce_sum(tokens)
    q.put((rank, t, u, float(first), list(sharding.split_sequences(5, rank, world)), passes, est, job))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_reduce_max_time_and_sum_units():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [11.0, 11.0]                 # max over ranks
    assert [r[2] for r in res] == [256.0, 256.0]               # 2 ranks x 2 sequences x 64 tokens
    assert res[0][3] != res[1][3]                              # ranks draw different data
    assert res[0][4] == [0, 1, 2] and res[1][4] == [3, 4]      # contiguous sequence blocks cover the batch
    assert res[0][5] == res[1][5] == [2.0, 5.0, 2.0]           # element-wise max over the ranks
    assert res[0][6] == res[1][6] == 6.0
    assert res[0][7] == res[1][7] == 256.0


def test_single_process_is_identity():
    assert sharding.reduce_job(3.5, 7.0) == (3.5, 7.0)
    w = workloads.configs()[0]
    assert sharding.rank_workload(w, 0, 1) is w
    assert sharding.rank_workload(w, 1, 2).seed == w.seed + 1000
    assert sharding.reduce_max_list([1.0, 2.0]) == [1.0, 2.0] and sharding.reduce_max(4.0) == 4.0
    assert sharding.reduce_sum(9.0) == 9.0
    assert [list(sharding.split_sequences(8, r, 4)) for r in range(4)] == [[0, 1], [2, 3], [4, 5], [6, 7]]
