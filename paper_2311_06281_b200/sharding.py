"""Multi-GPU plumbing.  Rows are independent sequences, so the path shards by rows with no
data-path collective: each rank runs the same kernels on its own rows.  The only communication is
the timing reduction (max over ranks) and a barrier, done with torch.distributed (NCCL on GPUs,
gloo in the CPU tests)."""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def shard_rows(rows: int, world: int, rank: int) -> tuple[int, int]:
    """Contiguous block of rows owned by `rank`: (first_row, row_count).  Blocks differ by at most one row."""
    if world < 1 or not (0 <= rank < world) or rows < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(rows, world)
    first = rank * base + min(rank, extra)
    return first, base + (1 if rank < extra else 0)


def init_from_env(backend: str | None = None) -> tuple[int, int, int]:
    """(rank, world, local_rank) from the torchrun environment; initialises the process group if world > 1."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        if backend is None:
            backend = "nccl" if torch.cuda.is_available() else "gloo"
        if backend == "nccl":
            torch.cuda.set_device(local)
            dist.init_process_group(backend, rank=rank, world_size=world, device_id=torch.device("cuda", local))
        else:
            dist.init_process_group(backend, rank=rank, world_size=world)
    return rank, world, local


def barrier():
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device="cpu") -> float:
    """Largest `value` over all ranks (the time of a multi-GPU step is its slowest rank's)."""
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device="cpu") -> float:
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())
