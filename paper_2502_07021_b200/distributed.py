"""Host-side plumbing for running the hot path on N GPUs of one node, one process per GPU.

The single-GPU path has no inter-GPU exchange, so N processes are N independent solvers, each on
its own problem instance (weak scaling: per-GPU work is fixed).  What the processes share is
only measurement: a barrier on both sides of the timed region, the MAX over ranks of the
device-timed duration, and the SUM of the units of work.  This module holds exactly that, on top
of ``torch.distributed`` (NCCL on GPUs, gloo on CPU for the tests).
"""
from __future__ import annotations

import os


def env_world():
    """(rank, local_rank, world_size) from the launcher's environment; (0, 0, 1) when absent."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str | None = None):
    """Join the process group if WORLD_SIZE > 1.  Returns (rank, local_rank, world_size)."""
    import torch
    import torch.distributed as dist
    rank, local_rank, world = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29511")
        if backend is None:
            backend = "nccl" if torch.cuda.is_available() else "gloo"
        if backend == "nccl":
            torch.cuda.set_device(local_rank)
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local_rank, world


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def aggregate(elapsed_ms: float, units: float, device=None):
    """(max over ranks of elapsed_ms, sum over ranks of units).  Identity for one process."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(elapsed_ms), float(units)
    if device is None:
        device = torch.device("cuda", torch.cuda.current_device()) if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([float(elapsed_ms)], dtype=torch.float64, device=device)
    u = torch.tensor([float(units)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def shard_problems(total: int, rank: int, world: int):
    """Contiguous share of `total` independent problems for `rank` (sizes differ by at most 1)."""
    base, extra = divmod(total, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def finalize():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()
