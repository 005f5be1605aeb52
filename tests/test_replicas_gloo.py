"""World-size-2 CPU test (gloo) of the replica plumbing used by bench.py --gpus N."""
import os
import socket
import sys

import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from paper_2411_11038_b200.replicas import Replicas
    r = Replicas(backend="gloo")
    r.barrier()
    slow = r.max_over_ranks(10.0 + 5.0 * rank)          # rank 1 is the slower replica
    thr = r.job_throughput(units_per_rank=3.0e12, ms=10.0 + 5.0 * rank)
    q.put((rank, r.world, slow, thr))
    r.barrier()
    r.close()


def test_two_replicas_take_the_slowest_time_and_add_their_work():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, world, slow, thr in got:
        assert world == 2 and slow == 15.0
        assert abs(thr - 2 * 3.0e12 / 15e-3) < 1e3


def test_single_process_needs_no_group():
    from paper_2411_11038_b200.replicas import Replicas
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        os.environ.pop(k, None)
    r = Replicas()
    assert r.world == 1 and r.max_over_ranks(3.5) == 3.5
    assert r.job_throughput(2.0, 1000.0) == 2.0
