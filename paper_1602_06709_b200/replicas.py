"""Host-side plumbing for running N independent replicas of the hot path, one
process per GPU (`bench.py --gpus N` under torchrun).  The path has no exchange
step on one node (the paper's multinode gradient exchange is out of scope), so
there is no data-path collective here: only a barrier around the timed region,
a max-over-ranks of the measured time, and a per-rank input shard id.
Works on the gloo backend too, which is how it is tested without GPUs."""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def world():
    return int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0"))


def init(backend: str, device=None):
    """Joins the process group when launched with WORLD_SIZE > 1; a no-op otherwise."""
    w, _, _ = world()
    if w > 1 and not dist.is_initialized():
        kwargs = {"device_id": device} if (device is not None and backend == "nccl") else {}
        dist.init_process_group(backend, **kwargs)
    return w


def barrier(cuda: bool):
    if dist.is_initialized():
        dist.barrier()
    if cuda:
        torch.cuda.synchronize()


def max_over_ranks(value: float, device="cpu") -> float:
    """The slowest rank's time is the job's time."""
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(units_per_rank_step: float, steps: int, n_ranks: int, slowest_ms: float) -> float:
    """Units all ranks processed divided by the slowest rank's time."""
    return units_per_rank_step * steps * n_ranks / (slowest_ms / 1e3)


def shutdown():
    if dist.is_initialized():
        dist.destroy_process_group()
