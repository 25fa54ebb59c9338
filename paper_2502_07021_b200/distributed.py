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


class _PhaseTimer:
    """Accumulates the time of the local device steps and of the exchanges of a sharded run: CUDA events on the
    shard's stream when there is one (read back after one synchronisation at the end), wall clock otherwise."""

    def __init__(self, stream, on_cuda):
        self.stream, self.on_cuda = stream, on_cuda
        self.marks, self.total = [], {"local": 0.0, "exchange": 0.0}

    def mark(self):
        import time

        import torch
        if self.on_cuda:
            ev = torch.cuda.Event(enable_timing=True)
            ev.record(self.stream)
            return ev
        return time.perf_counter()

    def add(self, phase, t0, t1):
        self.marks.append((phase, t0, t1))

    def result(self):
        if self.on_cuda and self.marks:
            self.marks[-1][2].synchronize()
        for phase, t0, t1 in self.marks:
            self.total[phase] += t0.elapsed_time(t1) if self.on_cuda else (t1 - t0) * 1e3
        self.marks = []
        return {"local_ms": self.total["local"], "exchange_ms": self.total["exchange"]}


def gather_blocks(local_block, sizes, out_full, group=None):
    """All-gather of contiguous blocks of unequal length (sizes[r] entries from rank r) into `out_full`, in rank
    order: every rank contributes its block padded to the longest one, and the valid parts are copied out."""
    import torch
    import torch.distributed as dist
    world = len(sizes)
    if not (dist.is_available() and dist.is_initialized()) or world == 1:
        out_full[:sizes[0]].copy_(local_block[:sizes[0]])
        return
    mmax = max(sizes)
    send = torch.zeros(mmax, dtype=local_block.dtype, device=local_block.device)
    send[:local_block.numel()].copy_(local_block)
    recv = [torch.empty(mmax, dtype=local_block.dtype, device=local_block.device) for _ in range(world)]
    dist.all_gather(recv, send, group=group)
    lo = 0
    for r in range(world):
        out_full[lo:lo + sizes[r]].copy_(recv[r][:sizes[r]])
        lo += sizes[r]


def sharded_iterate(api, shard, r_buf, k: int, stream=None, group=None, exchange: str = "allreduce", sizes=None,
                    timed: bool = False, fused_local: bool = True):
    """k Sinkhorn iterations of a row-partitioned problem, one shard per process.

    exchange = "allreduce": Algorithm 1 with the column sums assembled by ONE sum all-reduce of the per-shard
        partial products (n floats per iteration); valid for any K; the order of the additions is the
        collective library's.
    exchange = "ordered": the same partial products are all-gathered (G x n floats) and every shard adds them in
        rank order itself (fs_shard_col_finish_gathered): bit-reproducible whatever the library does.
    exchange = "alg1": Algorithm 1 as printed, two Allgathers of scaling slices per iteration, valid for a
        SYMMETRIC K (fs_shard_col_block_pass): the iterates are those of centralized Sinkhorn (Proposition 1).
        `sizes` lists the shards' row counts in rank order.

    `api` provides the fs_shard_* steps (the ctypes binding on GPUs); `r_buf` is a length-n float32 tensor on the
    shard's device.  Collectives are torch.distributed's (NCCL on GPUs, gloo on CPU); with a CUDA `stream` all
    steps are ordered on that stream.  With `fused_local` the row step and the column partial of the "allreduce" and
    "ordered" forms come from one read of the local block (fs_shard_fused_step) where that kernel applies.  With `timed` the time of the local steps and of the exchanges is
    accumulated separately (the paper's compute / communication split) and returned as a dict.
    """
    import contextlib

    import torch
    import torch.distributed as dist
    use_dist = dist.is_available() and dist.is_initialized()
    world = dist.get_world_size(group) if use_dist else 1
    rank = dist.get_rank(group) if use_dist else 0
    on_cuda = r_buf.is_cuda
    n = r_buf.numel()
    ctx = torch.cuda.stream(stream) if (stream is not None and on_cuda) else contextlib.nullcontext()
    timer = _PhaseTimer(stream, on_cuda and stream is not None) if timed else None

    def phase(name, fn):
        if timer is None:
            fn()
            return
        t0 = timer.mark()
        fn()
        timer.add(name, t0, timer.mark())

    with ctx:
        if exchange == "ordered":
            parts = torch.empty(world * n, dtype=r_buf.dtype, device=r_buf.device)
        if exchange == "alg1":
            if sizes is None:
                sizes = [row_range(n, r, world)[1] - row_range(n, r, world)[0] for r in range(world)]
            lo = sum(sizes[:rank])
            u_loc = torch.empty(sizes[rank], dtype=r_buf.dtype, device=r_buf.device)
            u_full = torch.empty(n, dtype=r_buf.dtype, device=r_buf.device)
            v_full = r_buf
        for _ in range(k):
            if exchange == "alg1":
                def local_u():
                    api.fs_shard_row_pass(shard, stream)
                    api.fs_shard_local_u(shard, u_loc, stream)
                phase("local", local_u)
                phase("exchange", lambda: gather_blocks(u_loc, sizes, u_full, group))
                v_loc = v_full[lo:lo + sizes[rank]]
                phase("local", lambda: api.fs_shard_col_block_pass(shard, u_full, v_loc, stream))
                phase("exchange", lambda: gather_blocks(v_loc.clone(), sizes, v_full, group))
                phase("local", lambda: api.fs_shard_set_scalings(shard, None, v_full, stream))
                continue

            def local_partial():
                # one read of the local block for both local steps where the fused kernel applies
                step = getattr(api, "fs_shard_fused_step", None) if fused_local else None
                if step is not None and step(shard, r_buf, stream, allow_unsupported=True):
                    return
                api.fs_shard_row_pass(shard, stream)
                api.fs_shard_col_partial(shard, r_buf, stream)
            phase("local", local_partial)
            if exchange == "ordered":
                def gather_parts():
                    if use_dist:
                        dist.all_gather(list(parts.view(world, n).unbind(0)), r_buf, group=group)
                    else:
                        parts[:n].copy_(r_buf)
                phase("exchange", gather_parts)
                phase("local", lambda: api.fs_shard_col_finish_gathered(shard, parts, world, n, stream))
            else:
                if use_dist:
                    phase("exchange", lambda: dist.all_reduce(r_buf, op=dist.ReduceOp.SUM, group=group))
                phase("local", lambda: api.fs_shard_col_finish(shard, r_buf, stream))
    return timer.result() if timer is not None else None


def finalize():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()
