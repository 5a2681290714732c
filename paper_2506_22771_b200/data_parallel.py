"""Data-parallel train step: the plumbing around ff_dp_train_phase.

The library cuts the step into phases at the points where the shards of a batch must exchange
data and says, after each phase, which device arrays to combine over the shards.  This module
holds what surrounds that: how a batch is split by rows, how a device address from the library
is turned back into a view of the torch tensor that owns it, and the all-reduce itself
(torch.distributed; NCCL on GPUs).  None of the method's arithmetic lives here."""
from __future__ import annotations

from typing import Callable, Iterable, List, Sequence, Tuple

from . import binding as ffb


def shard_rows(B_total: int, world: int, rank: int) -> Tuple[int, int]:
    """(row_offset, B_local) of a contiguous split of B_total rows per set over `world` shards; the
    first B_total % world shards hold one row more."""
    if world <= 0 or not 0 <= rank < world or B_total < world:
        raise ValueError("need 0 <= rank < world <= B_total")
    q, r = divmod(B_total, world)
    return rank * q + min(rank, r), q + (1 if rank < r else 0)


def shard_batch(X, B_total: int, row_offset: int, B_local: int):
    """Rows [row_offset, row_offset + B_local) of the positive and of the negative set of a batch laid
    out as [2 * B_total * rows_per_sample, features] (works for numpy arrays and torch tensors)."""
    per = X.shape[0] // (2 * B_total)
    pos = X[row_offset * per:(row_offset + B_local) * per]
    neg = X[(B_total + row_offset) * per:(B_total + row_offset + B_local) * per]
    if hasattr(X, "numpy") or not hasattr(X, "__array__"):
        import torch
        return torch.cat([pos, neg], 0)
    import numpy as np
    return np.concatenate([pos, neg], 0)


class PointerTable:
    """Maps a device (or host) address inside a registered torch tensor to a flat view of it."""

    def __init__(self, tensors: Iterable = ()):
        self._spans = []
        for t in tensors:
            self.add(t)

    def add(self, t):
        if t is not None:
            self._spans.append((t.data_ptr(), t.data_ptr() + t.numel() * t.element_size(), t))

    def add_layer_buffers(self, bufs: Sequence):
        for b in bufs:
            for t in (b.absmax, b.loss, b.accW_dump):
                self.add(t)

    def view(self, ptr: int, count: int, dtype: int):
        import torch
        want = torch.float32 if dtype == ffb.FF_DP_F32 else torch.int32
        for lo, hi, t in self._spans:
            if lo <= ptr and ptr + 4 * count <= hi:
                if t.dtype != want or (ptr - lo) % 4:
                    raise TypeError("the registered tensor does not hold that element type at that address")
                first = (ptr - lo) // 4
                return t.view(-1)[first:first + count]
        raise KeyError(f"address {ptr:#x} (+{4 * count} bytes) lies in no registered tensor")


def all_reduce_entries(entries: List[Tuple[int, int, int, int]], table: PointerTable, group=None):
    """Combines every listed array in place over the ranks of `group` (torch.distributed)."""
    import torch.distributed as dist
    for ptr, count, dtype, op in entries:
        v = table.view(ptr, count, dtype)
        dist.all_reduce(v, op=dist.ReduceOp.MAX if op == ffb.FF_DP_MAX else dist.ReduceOp.SUM, group=group)


def dp_train_step(ctx, descs_arr, bufs_arr, n_layers: int, B_local: int, B_total: int, row_offset: int, lam: float,
                  step: int, reduce: Callable[[List[Tuple[int, int, int, int]]], None], stream: int = 0):
    """All phases of one data-parallel step on this shard; `reduce(entries)` is called between phases
    and must combine the listed arrays over the shards, ordered after the phase on `stream`."""
    for phase in range(ffb.ff_dp_phase_count(n_layers)):
        entries = ffb.ff_dp_train_phase(ctx, descs_arr, bufs_arr, n_layers, B_local, B_total, row_offset, phase, lam,
                                        step, stream)
        if entries:
            reduce(entries)
