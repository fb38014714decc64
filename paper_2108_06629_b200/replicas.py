"""Aggregation of independent replicas (one process per GPU).

The training path does not shard: stages are streams of ONE GPU and there is no data-path
collective.  `bench.py --gpus N` therefore runs N independent replicas of the same job; the
only communication is the bookkeeping below -- a barrier around the timed region and a MAX
over ranks of the device-measured time -- done with torch.distributed (NCCL on GPUs, gloo in
the CPU tests).
"""


def max_over_ranks(value, dist=None, device="cpu"):
    """Largest `value` (a float) over all ranks; `dist` = torch.distributed or None for one rank."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replica_throughput(samples_per_replica, ms_local, dist=None, device="cpu"):
    """Whole-job samples/s of N replicas that each processed `samples_per_replica` samples:
    every replica counts, the slowest one sets the time."""
    world = 1 if dist is None or not dist.is_initialized() else dist.get_world_size()
    ms = max_over_ranks(ms_local, dist, device)
    return world * samples_per_replica / (ms * 1e-3), ms


def spawn_replicas(cmd, n, timeout=None, extra_env=None):
    """Run `cmd` (an argv list) as n replica processes, one per GPU, with the environment a launcher
    would give them (RANK, LOCAL_RANK, WORLD_SIZE, MASTER_ADDR = 127.0.0.1, a free MASTER_PORT),
    wait for all of them, and return what rank 0 wrote to its standard output.  Raises
    RuntimeError naming the first replica that failed."""
    import os
    import socket
    import subprocess
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        env.update(extra_env or {})
        procs.append(subprocess.Popen(cmd, env=env, stdout=subprocess.PIPE if r == 0 else subprocess.DEVNULL))
    out, failed = "", None
    for r, p in enumerate(procs):
        try:
            o, _ = p.communicate(timeout=timeout)
        except subprocess.TimeoutExpired:
            p.kill()
            o, _ = p.communicate()
            failed = failed if failed is not None else (r, "timed out")
        if r == 0 and o:
            out = o.decode()
        if p.returncode != 0 and failed is None:
            failed = (r, "exit code %s" % p.returncode)
    if failed is not None:
        for p in procs:
            if p.poll() is None:
                p.kill()
        raise RuntimeError("replica %d failed: %s" % failed)
    return out
