"""Multi-GPU bookkeeping of the measurement: the path runs as independent replicas, one process per GPU.

Sequences are independent, so N GPUs run N copies of the workload with no exchange on the data path; the
only collective work is the barrier around the timed region and the maximum of the per-rank times.  These
helpers hold that logic so that it can be exercised on CPU with the gloo backend.
"""
import torch
import torch.distributed as dist


def world_size():
    return dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1


def max_over_ranks(value, device="cpu"):
    """The slowest rank's value (a time): what a whole-job rate has to be computed from."""
    if world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank_per_step, ms_per_step):
    """Units per second over all replicas, from the slowest rank's time per step (weak scaling)."""
    return world_size() * units_per_rank_per_step / (ms_per_step * 1e-3)


def barrier():
    if world_size() > 1:
        dist.barrier()
