"""The N > 1 path of the benchmark is N independent replicas; what the ranks exchange is only
the timing bookkeeping.  Two gloo ranks on CPU check it: the slowest rank sets the time and
every rank's samples count."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2108_06629_b200 import replicas


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms_local = 10.0 if rank == 0 else 12.5            # rank 1 is slower
    value, ms = replicas.replica_throughput(2560, ms_local, dist)
    dist.barrier()
    out.put((rank, value, ms))
    dist.destroy_process_group()


def test_two_replicas_add_up_and_the_slowest_sets_the_time():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, value, ms in got:
        assert ms == 12.5
        assert abs(value - 2 * 2560 / 12.5e-3) < 1e-6


def test_single_rank_needs_no_process_group():
    value, ms = replicas.replica_throughput(100, 4.0, None)
    assert ms == 4.0 and abs(value - 25000.0) < 1e-9
