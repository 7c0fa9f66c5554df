"""Bookkeeping for running N independent replicas of the path, one process per GPU.

The attention path has no exchange step (requests are independent), so N > 1 means N replicas of the
workload.  This module only holds what the processes need to agree on a timing: rendezvous, a
barrier, the maximum of the ranks' elapsed times and the whole-job throughput.  The process group
is NCCL on GPUs and gloo on CPU (the tests)."""
from __future__ import annotations

import os
from typing import Optional, Tuple

import torch


def env_rank() -> Tuple[int, int, int]:
    """(rank, world size, local rank) from the environment torch.distributed.run sets."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def setup(backend: Optional[str] = None) -> Tuple[int, int, int]:
    rank, world, local = env_rank()
    if world > 1:
        import torch.distributed as dist
        if not dist.is_initialized():
            if backend is None:
                backend = "nccl" if torch.cuda.is_available() else "gloo"
            kw = {}
            if backend == "nccl":
                torch.cuda.set_device(local)
                kw["device_id"] = torch.device("cuda", local)
            dist.init_process_group(backend, **kw)
    return rank, world, local


def barrier(world: int) -> None:
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(x: float, world: int, device="cpu") -> float:
    if world == 1:
        return float(x)
    import torch.distributed as dist
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tokens_per_s(tokens_per_rank: int, elapsed_ms_this_rank: float, world: int, device="cpu") -> Tuple[float, float]:
    """Weak scaling: every rank processed `tokens_per_rank`; the job took as long as its slowest rank.
    Returns (tokens/s over all ranks, the slowest rank's milliseconds)."""
    ms = max_over_ranks(elapsed_ms_this_rank, world, device)
    return world * tokens_per_rank / (ms * 1e-3), ms


def shutdown() -> None:
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()
