"""Multi-GPU layout of the transform: replicas only.

The hot path is a single-GPU transform (the paper's core-to-core decomposition is out of scope), so
N GPUs run N independent cubes: rank r draws its own input (seed + r), nothing is exchanged on the data
path, and the only collective is the reduction of the timing (max over ranks).  These helpers hold that
logic so that it can be exercised with CPU processes (gloo) as well as on GPUs (nccl).
"""
import torch
import torch.distributed as dist


def rank_seed(base_seed, rank):
    """Seed of the cube rank `rank` transforms (distinct inputs per replica)."""
    return int(base_seed) + int(rank)


def max_over_ranks(value, device="cpu"):
    """Max of a scalar over all ranks of the default process group (identity without a group)."""
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank, ms_per_step_local, device="cpu"):
    """Whole-job throughput in units per second: all ranks' units over the slowest rank's time."""
    world = dist.get_world_size() if (dist.is_available() and dist.is_initialized()) else 1
    ms = max_over_ranks(ms_per_step_local, device)
    return world * units_per_rank / (ms * 1e-3), ms
