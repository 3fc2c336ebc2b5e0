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


# ---- the tensor-parallel form of the norm: all-reduce folded into the kernel ---------------------------------

@dataclass
class FusedAllreduceNorm:
    """One rank's view of a tensor-parallel group for the all-reduce-fused norm.

    ``x_parts[k]`` is rank k's partial x, ``y_outs[k]`` / ``r_outs[k]`` rank k's output tensors, all [n_rows, hidden]
    and all addressable from this rank's GPU (index ``rank`` is this rank's own memory, the others are peer
    mappings).  A call runs this rank's block of rows: it reads every rank's partial for those rows, and writes
    the rows of y into every rank's y, so that after all ranks' calls each rank holds all rows of y.  The new
    residual of those rows goes to this rank's own r_out only - the rank's next norm reads the residual of its
    own block and nothing else - unless ``gather_residual`` asks for every rank to receive it too.

    The kernel never waits for another rank.  The group meets in stream order instead: a one-element all-reduce
    on the launch stream before the kernel (every rank's partial is complete once it has run) and one after it
    (every rank's rows have been written once it has run).  Whatever produced this rank's partial must be ordered
    before the call on that same stream.  ``launch`` is
    ``binding.rmsnorm_allreduce_template_launch``; it is a parameter so that the host logic can run without a GPU.
    """
    rank: int
    world: int
    n_rows: int
    x_parts: list
    y_outs: list
    r_outs: list
    launch: object
    sync: object = None  # callable(stream) run before and after the launch; default: a one-element all-reduce on it
    gather_residual: bool = False
    _flag: object = None  # the meeting's one-element tensor, allocated once (no allocation per step)

    def __post_init__(self):
        if self.world not in (2, 4, 8):
            raise ValueError("the all-reduce-fused norm takes groups of 2, 4 or 8 ranks")
        if not (len(self.x_parts) == len(self.y_outs) == len(self.r_outs) == self.world):
            raise ValueError("one partial input and one pair of outputs per rank, in rank order")
        if not (0 <= self.rank < self.world):
            raise ValueError("rank outside the group")

    @property
    def shard(self) -> Shard:
        return strong_shard(self.n_rows, self.rank, self.world)

    def _meet(self, device, stream) -> None:
        """One meeting of the group, ordered on `stream` (None = the current stream): both the collective and the
        kernel between the two meetings must sit on one stream, or the kernel is ordered against neither."""
        if self.sync is not None:
            self.sync(stream)
            return
        if not dist.is_initialized():
            return
        if device.type == "cuda" and stream is not None:
            with torch.cuda.stream(stream):  # the collective is ordered against the stream that is current at the call
                if self._flag is None:
                    self._flag = torch.zeros(1, dtype=torch.int32, device=device)
                dist.all_reduce(self._flag)
        else:
            if self._flag is None:
                self._flag = torch.zeros(1, dtype=torch.int32, device=device)
            dist.all_reduce(self._flag)  # stream-ordered on NCCL: complete on the stream once every rank has reached it

    def __call__(self, theta, r, w, eps: float, stream=None) -> Shard:
        """r: this rank's residual [n_rows, hidden] (the same values on every rank); w: [hidden].  The two meetings
        and the launch between them are issued on `stream` (None: torch's current stream for all three)."""
        sh = self.shard
        self._meet(r.device, stream)
        r_outs = self.r_outs if self.gather_residual else [self.r_outs[self.rank]]
        self.launch(theta, self.x_parts, r, w, self.y_outs, r_outs, sh.row_begin, sh.rows, eps, stream)
        self._meet(r.device, stream)
        return sh


def gather_in_rank_order(obj) -> list:
    """Every rank's ``obj`` as a list indexed by rank (the list [obj] without a process group)."""
    if not dist.is_initialized():
        return [obj]
    out = [None] * dist.get_world_size()
    dist.all_gather_object(out, obj)
    return out


def symmetric_group_buffers(n_rows: int, hidden: int, dtype: torch.dtype, device: torch.device, names=("x", "y", "r_out")):
    """Allocate one [n_rows, hidden] tensor per name in symmetric memory and return, per name, the list of all
    ranks' tensors in rank order as seen from this GPU (own memory at this rank's index, peer mappings elsewhere).
    Needs an initialised NCCL process group whose ranks share one node."""
    import torch.distributed._symmetric_memory as symm_mem
    world, group = dist.get_world_size(), dist.group.WORLD
    out = {}
    for name in names:
        local = symm_mem.empty((n_rows, hidden), dtype=dtype, device=device)
        handle = symm_mem.rendezvous(local, group)
        out[name] = [local if k == dist.get_rank() else handle.get_buffer(k, (n_rows, hidden), dtype) for k in range(world)]
    return out


def fused_allreduce_norm(n_rows: int, hidden: int, dtype: torch.dtype, device: torch.device) -> FusedAllreduceNorm:
    """The group's buffers in symmetric memory, wired to the CUDA entry point.  Each rank writes its partial x into
    ``x_parts[rank]`` and reads the results from ``y_outs[rank]`` / ``r_outs[rank]``."""
    from . import binding
    bufs = symmetric_group_buffers(n_rows, hidden, dtype, device)
    return FusedAllreduceNorm(dist.get_rank(), dist.get_world_size(), n_rows, bufs["x"], bufs["y"], bufs["r_out"],
                              binding.rmsnorm_allreduce_template_launch)
