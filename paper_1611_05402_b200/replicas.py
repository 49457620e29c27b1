"""Aggregation of a run with N replicas (one process per GPU, no data-path collective).

The SGD path of the paper is specified on one device; with N ranks every rank runs its own replica
of the workload and only the timing meets: the job's time is the slowest rank's, the job's
throughput is all ranks' units over that time.
"""
import torch
import torch.distributed as dist


def slowest_rank_ms(ms_local, device):
    """Max over the ranks of a locally measured duration (milliseconds); identity without a process group."""
    ms = torch.tensor([float(ms_local)], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(ms, op=dist.ReduceOp.MAX)
    return float(ms.item())


def whole_job_value(units_per_rank, ms_local, device):
    """(value, ms): units of all ranks per second of the slowest rank, and that rank's milliseconds."""
    world = dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1
    ms = slowest_rank_ms(ms_local, device)
    return world * units_per_rank / (ms * 1e-3), ms
