"""Replica bookkeeping for runs on several GPUs of one node.

The verification step has no exchange between sequences, so N GPUs run N independent replicas of
the workload (one process per GPU).  The only thing the ranks share is timing: a job is as slow as
its slowest replica, so elapsed times are reduced with MAX, and throughput is the sum of the units
all replicas processed divided by that time.  No tensor of the hot path ever crosses ranks.
"""
import os

import torch


def world():
    """(rank, local_rank, world_size) from the launcher's environment (1 process = (0, 0, 1))."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend, device=None):
    """Join the job's process group (no-op for a single process); returns world_size."""
    _, _, n = world()
    if n > 1:
        import torch.distributed as dist
        if not dist.is_initialized():
            kw = {"device_id": torch.device(device)} if (device is not None and backend == "nccl") else {}
            dist.init_process_group(backend, **kw)
    return n


def barrier():
    _, _, n = world()
    if n > 1:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity for one process)."""
    _, _, n = world()
    if n == 1:
        return [float(v) for v in values]
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def aggregate_throughput(units_per_replica, seconds_per_step_each_rank, device="cpu"):
    """Whole-job units/s: all replicas' units over the slowest replica's time."""
    _, _, n = world()
    slowest = max_over_ranks([seconds_per_step_each_rank], device)[0]
    return n * units_per_replica / slowest, slowest


def shutdown():
    _, _, n = world()
    if n > 1:
        import torch.distributed as dist
        if dist.is_initialized():
            dist.destroy_process_group()
