"""Multi-process plumbing for replicated runs (one process per GPU).

The expert path on one GPU has no exchange step, so N GPUs run N independent replicas on
disjoint token batches; the only cross-rank traffic is the timing protocol: a barrier on
both sides of the timed region, the MAX over ranks of the elapsed time and the SUM of the
work done.  Works over NCCL (GPU) and gloo (CPU tests)."""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def init_from_env(backend: str | None = None):
    """-> (rank, world_size, local_rank); initialises the process group when WORLD_SIZE > 1."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        if backend is None:
            backend = "nccl" if torch.cuda.is_available() else "gloo"
        kw = {}
        if backend == "nccl":
            torch.cuda.set_device(local)
            kw["device_id"] = torch.device("cuda", local)
        dist.init_process_group(backend=backend, rank=rank, world_size=world, **kw)
    return rank, world, local


def _dev():
    if dist.is_initialized() and dist.get_backend() == "nccl":
        return torch.device("cuda", torch.cuda.current_device())
    return torch.device("cpu")


def barrier():
    if dist.is_initialized():
        dist.barrier()


def reduce_scalar(value: float, op: str) -> float:
    """MAX or SUM of a python float over all ranks (identity when single-process)."""
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=_dev())
    dist.all_reduce(t, op=dist.ReduceOp.MAX if op == "max" else dist.ReduceOp.SUM)
    return float(t.item())


def job_throughput(units_this_rank: float, seconds_this_rank: float) -> float:
    """Whole-job throughput: all ranks' units over the slowest rank's time."""
    total = reduce_scalar(units_this_rank, "sum")
    t = reduce_scalar(seconds_this_rank, "max")
    return total / t if t > 0 else 0.0


def shutdown():
    if dist.is_initialized():
        dist.destroy_process_group()
