"""The multi-process plumbing of the replicas-only multi-GPU mode, exercised on CPU with the gloo
backend at world size 2: rendezvous, barrier, MAX-over-ranks timing and the whole-job value."""
import os
import socket

import pytest
import torch
import torch.multiprocessing as mp

from paper_2606_01813_b200 import replicas


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    replicas.init_replicas("gloo")
    assert replicas.env_rank_world() == (rank, world, rank)
    replicas.barrier()
    local_ms = 10.0 + 5.0 * rank                     # rank 1 is the slow one
    mx = replicas.max_over_ranks(local_ms, torch.device("cpu"))
    value = replicas.whole_job_rounds_per_second(100, world, mx)
    seeds = [None] * world
    torch.distributed.all_gather_object(seeds, replicas.replica_seed(2000, rank))
    replicas.barrier()
    replicas.shutdown()
    out.put((rank, mx, value, seeds))


def test_two_replicas_gloo():
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
    for rank, mx, value, seeds in res:
        assert mx == pytest.approx(15.0)                         # the slowest rank decides
        assert value == pytest.approx(2 * 100 / 0.015)           # rounds of both ranks per second
        assert seeds == [2000, 2017] and len(set(seeds)) == world


def test_single_process_is_a_no_op():
    assert replicas.max_over_ranks(3.5, torch.device("cpu")) == 3.5
    assert replicas.whole_job_rounds_per_second(20, 1, 10.0) == pytest.approx(2000.0)
    replicas.barrier()
