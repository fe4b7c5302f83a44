"""The N>1 path is N independent replicas: ranks meet only to take the maximum elapsed time. Covered here
with two gloo ranks on CPU."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2511_11346_b200 import replicas


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, q):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    r, w = replicas.init_process_group("gloo")
    assert (r, w) == (rank, world) and replicas.rank_env() == (rank, rank, world)
    replicas.barrier()
    elapsed = 0.010 * (rank + 1)                     # rank 1 is the slow one
    slowest = replicas.max_over_ranks(elapsed)
    value = replicas.aggregate_throughput(8192, 5, w, slowest)
    q.put((rank, slowest, value, replicas.replica_seed_offset(rank)))
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank_and_the_summed_work():
    port = _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, slowest, value, _ in got:
        assert abs(slowest - 0.020) < 1e-12
        assert abs(value - 8192 * 5 * 2 / 0.020) < 1e-6
    assert got[0][3] != got[1][3]


def test_single_process_needs_no_process_group():
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        os.environ.pop(k, None)
    assert replicas.rank_env() == (0, 0, 1)
    assert replicas.max_over_ranks(1.5) == 1.5
    replicas.barrier()
    assert replicas.aggregate_throughput(100, 2, 1, 0.5) == 400.0
