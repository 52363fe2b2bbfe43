"""Replica bookkeeping for runs on several GPUs.

A SPACE step (Algorithm 1: block attention, verification, KV commit) of one
batch never exchanges data with another batch, so several GPUs run independent
replicas: one process per GPU, every rank with its own seeded input sets, and
no collective on the data path.  The only exchange is the timing reduction
below: the job's time is the slowest rank's, its throughput the steps of all
ranks over that time.
"""
import os

import torch
import torch.distributed as dist

SETS_PER_RANK = 1000   # input-set indices [rank * SETS_PER_RANK, (rank + 1) * SETS_PER_RANK) belong to a rank


def rank_env():
    """(rank, world size, local rank) as the launcher exported them; (0, 1, 0) without a launcher."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def set_index(rank, i):
    """Index of rank `rank`'s i-th input set: distinct ranks never share a set."""
    if not 0 <= i < SETS_PER_RANK:
        raise ValueError(f"a rank owns {SETS_PER_RANK} input sets, asked for set {i}")
    return rank * SETS_PER_RANK + i


def init(backend, local_rank=0):
    """Join the process group when a launcher started several ranks; returns the world size."""
    _, world, _ = rank_env()
    if world > 1 and not dist.is_initialized():
        if backend == "nccl":
            dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        else:
            dist.init_process_group(backend)
    return world


def barrier():
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def slowest(seconds, device="cpu"):
    """Maximum of a per-rank duration over all ranks (the value itself on one rank)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(seconds)
    t = torch.tensor([float(seconds)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(steps_per_rank, seconds_local, device="cpu"):
    """Whole-job steps per second: every rank ran `steps_per_rank` steps; the job took the slowest rank's time."""
    world = dist.get_world_size() if (dist.is_available() and dist.is_initialized()) else 1
    t = slowest(seconds_local, device)
    return world * steps_per_rank / t, t


def shutdown():
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()
