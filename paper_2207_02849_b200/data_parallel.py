"""Row-sharded data-parallel use of the library (Sec. 4 of the paper lists data-parallel training among the
systems features; App. E reports it on 2 GPUs): one process and one GPU per rank, the rows of every batch
partitioned over the ranks, parameters and solver state replicated, one all-reduce (sum) of a vector per
gradient / Hessian-vector product / mixed product.  Only plumbing lives here: which rows a rank holds, its
weight, and the all-reduce itself through torch.distributed (NCCL for device buffers, gloo for host ones).
The arithmetic stays in the CUDA library, which calls back into `DeviceAllReduce` between its kernels."""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_rows(n: int, rank: int, world: int) -> tuple[int, int]:
    """Half-open row range [lo, hi) of rank `rank`: contiguous, disjoint, covering 0..n, sizes differing by
    at most one row."""
    if not (0 <= rank < world):
        raise ValueError("rank outside the job")
    return (n * rank) // world, (n * (rank + 1)) // world


def row_weight(n: int, rank: int, world: int) -> float:
    """Share of the rows rank `rank` holds; the weights of all ranks sum to one."""
    lo, hi = shard_rows(n, rank, world)
    return (hi - lo) / float(n) if n > 0 else 1.0 / world


def allreduce_sum_(t: torch.Tensor, group=None) -> torch.Tensor:
    """In-place sum of a tensor over the ranks of `group` (host tensors: gloo; device tensors: NCCL)."""
    if dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
    return t


class _RawDeviceBuffer:
    """fp32 device memory at a raw address, exposed through the CUDA array interface so that torch can view
    it without owning it."""

    def __init__(self, ptr: int, count: int):
        self.__cuda_array_interface__ = {"shape": (count,), "typestr": "<f4", "data": (ptr, False), "version": 3,
                                         "strides": None}


class DeviceAllReduce:
    """The callable a data-parallel `Level` hands to the library: sums `count` floats at a device address
    over the ranks, ordered on the stream the library is enqueuing on."""

    def __init__(self, group=None, single_rank_too: bool = False):
        """single_rank_too: issue the collective even in a job of one rank (it then changes nothing; useful to
        exercise the exchange itself on one GPU)."""
        self.group = group
        self.single_rank_too = single_rank_too
        self.calls = 0
        self.floats = 0

    def __call__(self, ptr: int, count: int, stream: int) -> None:
        self.calls += 1
        self.floats += count
        if not dist.is_initialized() or (dist.get_world_size(self.group) <= 1 and not self.single_rank_too):
            return
        t = torch.as_tensor(_RawDeviceBuffer(ptr, count), device=torch.device("cuda", torch.cuda.current_device()))
        with torch.cuda.stream(torch.cuda.ExternalStream(stream) if stream else torch.cuda.default_stream()):
            dist.all_reduce(t, op=dist.ReduceOp.SUM, group=self.group)


def shard_level(level, n_global: int, rank: int, world: int, allreduce) -> None:
    """Declares `level` (already built on this rank's rows only) to be rank `rank`'s share of a batch of
    n_global rows."""
    level.set_comm(allreduce, row_weight(n_global, rank, world))
