"""Multi-GPU plumbing: independent replicas, one process per GPU.

The decode path has no exchange step: every (sequence, KV head) unit owns its blocks, statistics, state,
selection and output.  N GPUs therefore run N independent replicas of the workload (weak scaling) and the only
communication is what a measurement needs: a barrier around the timed region and the maximum of the ranks'
device times.  The same code runs over `gloo` on CPU, which is how it is tested.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_world():
    """(world_size, rank, local_rank) as the launcher exports them; (1, 0, 0) without a launcher."""
    return (int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init(backend: str, device=None):
    """Joins the process group when there is more than one rank.  Returns (world_size, rank)."""
    world, rank, _ = env_world()
    if world > 1 and not dist.is_initialized():
        if backend == "nccl":
            dist.init_process_group("nccl", device_id=torch.device(device))
        else:
            dist.init_process_group(backend)
    return world, rank


def barrier(device=None):
    if dist.is_initialized():
        dist.barrier()
    if device is not None and torch.device(device).type == "cuda":
        torch.cuda.synchronize(device)


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum over the ranks of a list of floats (each rank's own device times)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_initialized():
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def whole_job_rate(units_per_rank_per_step: int, steps: int, ms_max: float) -> float:
    """Units per second of the whole job: every rank does the same work; the slowest rank sets the time."""
    world = dist.get_world_size() if dist.is_initialized() else 1
    return units_per_rank_per_step * world * steps / (ms_max * 1e-3)


def shutdown():
    if dist.is_initialized():
        dist.destroy_process_group()
