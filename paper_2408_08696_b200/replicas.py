"""Multi-GPU runs are independent replicas (the step has no exchange between GPUs): every rank times its own
loop and the job's time is the slowest rank's.  Works with any torch.distributed backend (nccl on GPUs, gloo
on CPU for tests)."""
from __future__ import annotations

import torch
import torch.distributed as dist


def world():
    if dist.is_available() and dist.is_initialized():
        return dist.get_rank(), dist.get_world_size()
    return 0, 1


def barrier():
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(value, device="cpu"):
    """Largest `value` (a float) over all ranks; identity without a process group."""
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def max_over_ranks_vec(values, device="cpu"):
    """Element-wise largest value over all ranks of a list of floats (one entry per timed block)."""
    if not (dist.is_available() and dist.is_initialized()):
        return [float(v) for v in values]
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def aggregate(elapsed_ms, steps_per_rank, device="cpu", reduce=True):
    """Whole-job figures for `world` replicas that each ran `steps_per_rank` steps in `elapsed_ms` (this rank's
    device time, or with reduce=False a time that already is the maximum over ranks): the job takes the slowest
    rank's time and completes world * steps_per_rank steps."""
    _, n = world()
    t_ms = max_over_ranks(elapsed_ms, device) if reduce else float(elapsed_ms)
    total_steps = n * steps_per_rank
    return {
        "n_ranks": n,
        "ms_per_step": t_ms / steps_per_rank,                 # one step of every replica, side by side
        "us_per_step_job": 1000.0 * t_ms / total_steps,       # job time per completed step
        "steps_per_s": total_steps / (t_ms / 1000.0),
    }
