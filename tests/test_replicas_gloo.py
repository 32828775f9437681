"""The N > 1 path of the benchmark (independent replicas, barrier, MAX over ranks, whole-job rate)
on two gloo ranks on CPU."""
import os
import socket

import torch
import torch.multiprocessing as mp


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_2511_16786_b200 import replicas
    assert replicas.world_from_env() == (rank, world, rank)
    dist = replicas.init("gloo")
    assert dist is not None and dist.get_world_size() == world
    replicas.barrier(dist)
    mine = 10.0 + 5.0 * rank                       # rank 1 is the slow one
    slowest = replicas.max_over_ranks(mine, dist)
    rate = replicas.whole_job_rate(32768, world, slowest)
    out.put((rank, slowest, rate))
    replicas.barrier(dist)
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
    for rank, slowest, rate in res:
        assert slowest == 15.0
        assert abs(rate - 32768 * 2 / 0.015) < 1e-6


def test_single_process_needs_no_group():
    from paper_2511_16786_b200 import replicas
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        os.environ.pop(k, None)
    assert replicas.init("gloo") is None
    assert replicas.max_over_ranks(3.5, None) == 3.5
    assert replicas.whole_job_rate(100, 1, 1000.0) == 100.0
