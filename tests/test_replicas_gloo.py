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


_STUB = r"""
import json, os, sys
sys.path.insert(0, %r)
import torch.distributed as dist
from paper_2108_06629_b200 import replicas
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
assert int(os.environ["LOCAL_RANK"]) == rank and os.environ["MASTER_ADDR"] == "127.0.0.1"
dist.init_process_group("gloo", rank=rank, world_size=world)
value, ms = replicas.replica_throughput(1000, 5.0 + rank, dist)      # the last rank is the slowest
dist.barrier()
if rank == 0:
    print(json.dumps({"n_gpus": world, "value": value, "ms": ms}))
dist.destroy_process_group()
if os.environ.get("LP_STUB_FAIL_RANK") == str(rank):
    sys.exit(3)
"""


def test_spawned_replicas_get_a_launchers_environment_and_rank_zero_reports():
    """`bench.py --gpus N` started without a launcher spawns its N replicas through
    replicas.spawn_replicas; here the replicas are a CPU stub over gloo."""
    import json
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = replicas.spawn_replicas([sys.executable, "-c", _STUB % root], 3, timeout=180)
    line = json.loads(out.strip().splitlines()[-1])
    assert line["n_gpus"] == 3 and line["ms"] == 7.0
    assert abs(line["value"] - 3 * 1000 / 7.0e-3) < 1e-6


def test_a_failing_replica_is_reported():
    import sys
    import pytest
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    with pytest.raises(RuntimeError, match="replica 1 failed"):
        replicas.spawn_replicas([sys.executable, "-c", _STUB % root], 2, timeout=180, extra_env={"LP_STUB_FAIL_RANK": "1"})


def test_bench_hands_gpus_n_to_the_spawner(monkeypatch, capsys):
    """Without WORLD_SIZE in the environment, `--gpus 2` must go through the spawner with the same
    command line (and with it, under a launcher, must not)."""
    import importlib
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    sys.path.insert(0, root)
    bench = importlib.import_module("bench")
    seen = {}

    def fake(cmd, n, **kw):
        seen["cmd"], seen["n"] = cmd, n
        return '{"n_gpus": 2}\n'
    monkeypatch.setattr(bench.replicas, "spawn_replicas", fake)
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "2", "--steps", "3", "--workload", "mlp4_784"])
    bench.main()
    assert seen["n"] == 2 and seen["cmd"][-6:] == ["--gpus", "2", "--steps", "3", "--workload", "mlp4_784"]
    assert capsys.readouterr().out.strip() == '{"n_gpus": 2}'
