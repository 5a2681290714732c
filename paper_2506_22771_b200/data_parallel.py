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


SMALL = 64   # entries of at most this many elements are packed into one collective per (type, operation)


def _torch_op(op: int):
    import torch.distributed as dist
    return dist.ReduceOp.MAX if op == ffb.FF_DP_MAX else dist.ReduceOp.SUM


def all_reduce_entries(entries: List[Tuple], table: PointerTable, group=None):
    """Combines every listed array in place over the ranks of `group` (torch.distributed), in stream order.  The
    small entries of a phase (ranges, loss shares) share one collective per element type and operation: they are
    packed into a staging tensor, reduced together and copied back - a phase costs one or two latencies instead of
    one per entry."""
    import torch
    import torch.distributed as dist
    if dist.get_world_size(group) == 1:
        return                       # one shard: every array already is the whole batch's
    packs = {}
    for ent in entries:
        ptr, count, dtype, op = ent[:4]
        v = table.view(ptr, count, dtype)
        if count <= SMALL:
            packs.setdefault((dtype, op), []).append(v)
        else:
            dist.all_reduce(v, op=_torch_op(op), group=group)
    for (dtype, op), views in packs.items():
        if len(views) == 1:
            dist.all_reduce(views[0], op=_torch_op(op), group=group)
            continue
        staged = torch.cat([v.reshape(-1) for v in views])
        dist.all_reduce(staged, op=_torch_op(op), group=group)
        at = 0
        for v in views:
            v.copy_(staged[at:at + v.numel()].reshape(v.shape))
            at += v.numel()


class OverlappedReducer:
    """The reductions of a data-parallel step with the large ones taken off the critical path.

    now(entries): combine at once, in stream order (small entries packed as in all_reduce_entries).
    start(entries) -> handle: begin combining on a side stream, ordered after everything enqueued so far on the
    compute stream (an event); finish(handle): make the compute stream wait for it.  On CPU tensors (the gloo tests)
    there are no streams: start issues the collectives with async_op=True and finish waits for them."""

    def __init__(self, table: PointerTable, group=None, device=None):
        self.table, self.group = table, group
        self.cuda = device is not None and str(device).startswith("cuda")
        self.side = None
        self.log = []              # ("now" | "start" | "finish", phase tag) in call order, for the tests
        if self.cuda:
            import torch
            self.side = torch.cuda.Stream(device=device)

    def now(self, entries, tag=None):
        self.log.append(("now", tag))
        all_reduce_entries(entries, self.table, self.group)

    def start(self, entries, tag=None):
        import torch
        import torch.distributed as dist
        self.log.append(("start", tag))
        if dist.get_world_size(self.group) == 1:
            return ("none", None, None)
        views = [self.table.view(*e[:3]) for e in entries]
        if self.cuda:
            ready = torch.cuda.Event()
            ready.record(torch.cuda.current_stream())
            self.side.wait_event(ready)
            with torch.cuda.stream(self.side):
                for v, e in zip(views, entries):
                    dist.all_reduce(v, op=_torch_op(e[3]), group=self.group)
                done = torch.cuda.Event()
                done.record(self.side)
            return ("event", done, views)
        works = [dist.all_reduce(v, op=_torch_op(e[3]), group=self.group, async_op=True) for v, e in zip(views, entries)]
        return ("works", works, views)

    def finish(self, handle, tag=None):
        import torch
        self.log.append(("finish", tag))
        kind, obj, _views = handle
        if kind == "none":
            return
        if kind == "event":
            torch.cuda.current_stream().wait_event(obj)
        else:
            for w in obj:
                w.wait()


def dp_train_step(ctx, descs_arr, bufs_arr, n_layers: int, B_local: int, B_total: int, row_offset: int, lam: float,
                  step: int, reduce, stream: int = 0):
    """All phases of one data-parallel step on this shard.

    `reduce` is either a callable reduce(entries) that combines the listed arrays over the shards in stream order
    (every reduction then sits between its phase and the next), or an object with now / start / finish like
    OverlappedReducer: a reduction whose result is needed only several phases later (the INT32 weight-gradient
    sums of a layer, read by that layer's update phase) is started behind its phase and waited for just before
    the phase that needs it, so it runs beside the contractions of the layers after it."""
    overlapped = hasattr(reduce, "start")
    pending = {}                                   # phase that needs the result -> handles
    for phase in range(ffb.ff_dp_phase_count(n_layers)):
        for h in pending.pop(phase, []):
            reduce.finish(h, phase)
        entries = ffb.ff_dp_train_phase(ctx, descs_arr, bufs_arr, n_layers, B_local, B_total, row_offset, phase, lam,
                                        step, stream)
        if not entries:
            continue
        if not overlapped:
            reduce(entries)
            continue
        soon = [e for e in entries if e[4] <= phase + 1]
        later = [e for e in entries if e[4] > phase + 1]
        if soon:
            reduce.now(soon, phase)
        for need in sorted({e[4] for e in later}):
            pending.setdefault(need, []).append(reduce.start([e for e in later if e[4] == need], phase))
    assert not pending, "a reduction was asked for by a phase that does not exist"
