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
