"""The N > 1 path of the benchmark (independent replicas, max-over-ranks timing) on two CPU ranks over gloo."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2001_00138_b200 import replicas


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms, e2e = replicas.max_over_ranks([3.0 + rank, 10.0 - rank])
        lo, hi = replicas.shard_batch(65, world, rank)
        t = torch.tensor([hi - lo], dtype=torch.int64)
        dist.all_reduce(t)
        out.put((rank, ms, e2e, lo, hi, int(t)))
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, e2e, lo, hi, total in res:
        assert ms == 4.0 and e2e == 10.0          # both ranks agree on the maximum
        assert total == 65
    assert [(r[3], r[4]) for r in res] == [(0, 33), (33, 65)]
    assert replicas.whole_job_value(100.0, 2.0, 2) == 100.0


def test_single_process_is_the_identity():
    assert replicas.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert replicas.shard_batch(7, 3, 2) == (5, 7)
    with pytest.raises(ValueError):
        replicas.shard_batch(4, 2, 2)
