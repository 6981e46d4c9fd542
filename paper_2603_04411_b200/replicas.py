"""Replica bookkeeping for runs on several GPUs.

The hot path has no exchange step (sequences are independent), so N GPUs run N replicas of the
workload and nothing crosses the links on the data path.  What the ranks do share is the timing
protocol: a barrier on both sides of the timed region, the MAXIMUM over ranks of every device time,
and a whole-job throughput = the units all ranks processed / that maximum.  The process group is
NCCL on GPUs; the same code runs on gloo in the CPU tests.
"""
import os

import torch
import torch.distributed as dist


def world_size() -> int:
    return int(os.environ.get("WORLD_SIZE", "1"))


def rank() -> int:
    return int(os.environ.get("RANK", "0"))


def init(backend: str, device=None) -> None:
    """Joins the process group described by RANK / WORLD_SIZE / MASTER_ADDR / MASTER_PORT (no-op for one rank)."""
    if world_size() > 1 and not dist.is_initialized():
        if backend == "nccl":
            dist.init_process_group("nccl", device_id=device)
        else:
            dist.init_process_group(backend)


def barrier() -> None:
    if world_size() > 1:
        dist.barrier()


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum over all ranks of a list of floats (every rank gets the result)."""
    t = torch.tensor([float(x) for x in values], dtype=torch.float64, device=device)
    if world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.tolist()]


def whole_job_rate(units_per_rank: float, ms: float) -> float:
    """Units per second of the whole job: every rank processed units_per_rank units in `ms` (already the max over ranks)."""
    return world_size() * units_per_rank / (ms * 1e-3)


def finish() -> None:
    if world_size() > 1 and dist.is_initialized():
        dist.destroy_process_group()
