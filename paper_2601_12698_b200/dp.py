"""Data-parallel plumbing: rows are independent, so N GPUs are N row shards with `w` replicated.

There is no data-path collective.  The only communication is control: a barrier around the timed
region, the maximum of the per-rank times, and a broadcast of the chosen theta from rank 0.  These work
over any torch.distributed backend (NCCL on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

import os
from dataclasses import dataclass

import torch
import torch.distributed as dist


@dataclass(frozen=True)
class Shard:
    rank: int
    world: int
    row_begin: int  # first global row owned by this rank
    row_end: int    # one past the last

    @property
    def rows(self) -> int:
        return self.row_end - self.row_begin


def env_world() -> tuple[int, int, int]:
    """(rank, world_size, local_rank) from the launcher's environment; (0, 1, 0) when run plainly."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def weak_shard(rows_per_rank: int, rank: int, world: int) -> Shard:
    """Weak scaling: every rank owns `rows_per_rank` rows of a job of world * rows_per_rank rows."""
    if not (0 <= rank < world) or rows_per_rank < 0:
        raise ValueError("bad shard request")
    return Shard(rank, world, rank * rows_per_rank, (rank + 1) * rows_per_rank)


def strong_shard(total_rows: int, rank: int, world: int) -> Shard:
    """Strong scaling: a fixed job split into contiguous blocks whose sizes differ by at most one row."""
    if not (0 <= rank < world) or total_rows < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(total_rows, world)
    begin = rank * base + min(rank, extra)
    return Shard(rank, world, begin, begin + base + (1 if rank < extra else 0))


def init(backend: str | None = None, device: torch.device | None = None) -> bool:
    """Join the process group when launched with WORLD_SIZE > 1.  Returns True when distributed."""
    _, world, _ = env_world()
    if world <= 1:
        return False
    if not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        kwargs = {}
        if device is not None and device.type == "cuda":
            kwargs["device_id"] = device
        dist.init_process_group(backend or ("nccl" if torch.cuda.is_available() else "gloo"), **kwargs)
    return True


def barrier(device: torch.device) -> None:
    if dist.is_initialized():
        if device.type == "cuda":
            dist.barrier(device_ids=[device.index])
        else:
            dist.barrier()
    if device.type == "cuda":
        torch.cuda.synchronize(device)


def max_over_ranks(value: float, device: torch.device) -> float:
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device: torch.device) -> float:
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def broadcast_ints(values: list[int], device: torch.device, src: int = 0) -> list[int]:
    if not dist.is_initialized():
        return list(values)
    t = torch.tensor(values, dtype=torch.int64, device=device)
    dist.broadcast(t, src=src)
    return [int(v) for v in t.tolist()]


def whole_job_rate(units_per_rank_per_step: float, steps: int, world: int, max_ms: float) -> float:
    """Units per second of the whole job: all ranks' work over the slowest rank's time."""
    return units_per_rank_per_step * steps * world / (max_ms * 1e-3)


def shutdown() -> None:
    if dist.is_initialized():
        dist.destroy_process_group()
