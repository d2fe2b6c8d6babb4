"""The N > 1 leg of the bench on CPU: two gloo ranks, each with its own batch, timings reduced by
max and tokens by sum - the only cross-rank traffic of the path (it has no data-path collective)."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench
from paper_2609_32999_b200 import binding as tb


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = bench.rank_workload(3, rank, requests=2)
    plan = tb.Plan(w, host_only=True)                 # host placement of this rank's shard
    assert plan.info.total_tokens == w.total_tokens
    times, tokens = bench.aggregate([10.0 + rank, 3.0 - rank], w.total_tokens, world, "cpu")
    all_tok = [None] * world
    dist.all_gather_object(all_tok, (int(w.total_tokens), w.unit_pages[:4].tolist()))
    if rank == 0:
        out.put((times, tokens, all_tok))
    dist.destroy_process_group()


def test_two_ranks_shard_by_request_and_reduce():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    times, tokens, all_tok = q.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert times == [11.0, 3.0]                                   # max over ranks of each timing
    assert tokens == float(all_tok[0][0] + all_tok[1][0])         # whole-job tokens
    assert all_tok[0] != all_tok[1]                               # ranks drew different batches


def test_single_rank_aggregate_is_identity():
    times, tokens = bench.aggregate([1.5, 2.5], 42, 1, "cpu")
    assert times == [1.5, 2.5] and tokens == 42.0
    a, b = bench.rank_workload(4, 0, requests=1), bench.rank_workload(4, 1, requests=1)
    assert a.total_tokens == b.total_tokens == 33024 and not np.array_equal(a.unit_pages, b.unit_pages)
