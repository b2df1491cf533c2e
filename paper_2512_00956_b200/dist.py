"""Process-group plumbing for the benchmark: one process per GPU, no data-path collective.

The online layer shards over tokens (rows of X are independent, Eq. 7), so N GPUs run N
replicas on their own token batches ("weak" scaling); the only communication is the
barrier around the timed region and a MAX-reduction of the per-rank device time.
"""
import os

import torch
import torch.distributed as dist


def env_world():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def init(backend=None):
    rank, local_rank, world = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29512")
        if backend is None:
            backend = "nccl" if torch.cuda.is_available() else "gloo"
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local_rank, world


def barrier():
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(value, device="cpu"):
    """MAX of a python float over all ranks (identity when not distributed)."""
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value, device="cpu"):
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def whole_job_rate(units_this_rank, seconds_this_rank, device="cpu"):
    """Aggregate throughput: units processed by all ranks / slowest rank's time."""
    t = max_over_ranks(seconds_this_rank, device)
    u = sum_over_ranks(units_this_rank, device)
    return u / t, t


def shutdown():
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()
