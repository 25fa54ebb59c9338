"""Host-side plumbing for running the hot path on N GPUs of one node, one process per GPU.

The single-GPU path has no inter-GPU exchange, so N processes are N independent solvers, each on
its own problem instance (weak scaling: per-GPU work is fixed).  What the processes share there
is only measurement: a barrier on both sides of the timed region, the MAX over ranks of the
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


def row_range(n: int, rank: int, world: int):
    """Contiguous rows [lo, hi) of an n x n problem owned by `rank` (the paper's index set I_rank)."""
    return shard_problems(n, rank, world)


def sharded_iterate(api, shard, r_buf, k: int, stream=None, group=None):
    """k Sinkhorn iterations of a row-partitioned problem, one shard per process (Algorithm 1 with the
    column sums assembled by an all-reduce of the per-shard partial products, n floats per iteration).

    `api` provides fs_shard_row_pass / fs_shard_col_partial / fs_shard_col_finish (the ctypes binding on
    GPUs); `r_buf` is a length-n float32 tensor on the shard's device that receives the partial and then
    the reduced column sums.  The collective is torch.distributed's (NCCL on GPUs, gloo on CPU); with a
    CUDA `stream` the three steps and the collective are ordered on that stream.
    """
    import contextlib

    import torch
    import torch.distributed as dist
    use_dist = dist.is_available() and dist.is_initialized()
    ctx = torch.cuda.stream(stream) if (stream is not None and r_buf.is_cuda) else contextlib.nullcontext()
    with ctx:
        for _ in range(k):
            api.fs_shard_row_pass(shard, stream)
            api.fs_shard_col_partial(shard, r_buf, stream)
            if use_dist:
                dist.all_reduce(r_buf, op=dist.ReduceOp.SUM, group=group)
            api.fs_shard_col_finish(shard, r_buf, stream)


def finalize():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()
