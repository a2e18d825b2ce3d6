"""A symmetric heap over the ranks of a torch.distributed group: the host side of Section 3.2's initialisation.

Every rank allocates its own slot, exports a handle to it, the handles are all-gathered, every rank opens its
peers' slots and builds the table of bases that the kernels translate pointers with (Section 3.3).  The slot of
rank r then has one address per process; offsets inside a slot are the same everywhere (symmetric allocation).

This module only orders calls of the C-ABI library (binding.py) and of torch.distributed; nothing here
computes.  The memory operations are injected (`ops`) so that the exchange can be exercised without a GPU.
"""
from __future__ import annotations

from . import binding as _b


class CudaOps:
    """The library's own allocation / export / open / heap calls."""

    alloc = staticmethod(_b.iris_ipc_alloc)
    free = staticmethod(_b.iris_ipc_free)
    export = staticmethod(_b.iris_ipc_export)
    open = staticmethod(_b.iris_ipc_open)
    close = staticmethod(_b.iris_ipc_close)
    heap_create = staticmethod(_b.iris_heap_create_from_bases)
    heap_destroy = staticmethod(_b.iris_heap_destroy)


def exchange_bases(local_ptr: int, handle: bytes, rank: int, world: int, all_gather, open_handle) -> tuple[list[int], list[int]]:
    """bases[r] for every rank r, and the peer mappings this call opened.

    all_gather(obj) -> list of every rank's obj in rank order; open_handle(bytes) -> address in this process.
    A rank never opens its own handle (the runtime refuses that): its own entry is the local allocation.
    """
    if not 0 <= rank < world:
        raise ValueError(f"rank {rank} outside [0, {world})")
    entries = all_gather((rank, bytes(handle)))
    if len(entries) != world:
        raise RuntimeError(f"all-gather returned {len(entries)} entries for {world} ranks")
    bases: list[int] = [0] * world
    opened: list[int] = []
    for pos, (r, hd) in enumerate(entries):
        if r != pos:
            raise RuntimeError(f"all-gather entry {pos} comes from rank {r}: not in rank order")
        if r == rank:
            bases[r] = local_ptr
        else:
            p = open_handle(hd)
            bases[r] = p
            opened.append(p)
    if len(set(bases)) != world or any(b == 0 for b in bases):
        raise RuntimeError("a slot is missing or mapped twice")
    return bases, opened


class DistributedHeap:
    """One rank's view of the heap.  `handle` is what the C-ABI calls take; `bases[r]` is rank r's slot here.

    Collective: every rank of `group` constructs it with the same bytes_per_rank, and closes it, at the same
    point of the program.  The constructor ends with a barrier, so that no rank launches into a slot that its
    owner has not allocated and cleared yet; close() starts with one, so that no rank releases a slot that a
    peer's kernels still write.
    """

    def __init__(self, bytes_per_rank: int, group=None, ops=None, dist=None):
        if dist is None:
            import torch.distributed as dist
        self._dist, self._group = dist, group
        self._ops = ops if ops is not None else CudaOps
        self.rank = dist.get_rank(group)
        self.world = dist.get_world_size(group)
        if self.world > _b.IRIS_MAX_WORLD:
            raise ValueError(f"world {self.world} exceeds IRIS_MAX_WORLD = {_b.IRIS_MAX_WORLD}")
        if bytes_per_rank <= 0 or bytes_per_rank % 256:
            raise ValueError("bytes_per_rank must be a positive multiple of 256")
        self.bytes_per_rank = bytes_per_rank
        self.handle = None
        self._opened: list[int] = []
        self._local = self._ops.alloc(bytes_per_rank)
        try:
            hd = self._ops.export(self._local)

            def all_gather(obj):
                out = [None] * self.world
                dist.all_gather_object(out, obj, group=group)
                return out

            self.bases, self._opened = exchange_bases(self._local, hd, self.rank, self.world, all_gather, self._ops.open)
            self.handle = self._ops.heap_create(self.world, bytes_per_rank, self.bases, self.rank)
        except Exception:
            self._release()
            raise
        dist.barrier(group=group)

    def _release(self):
        if self.handle is not None:
            self._ops.heap_destroy(self.handle)
            self.handle = None
        for p in self._opened:
            self._ops.close(p)
        self._opened = []
        if self._local:
            self._ops.free(self._local)
            self._local = 0

    def barrier(self):
        """Host barrier over the group; the caller synchronises its device first when kernels are in flight."""
        self._dist.barrier(group=self._group)

    def close(self):
        """Collective.  Peer mappings are closed before any owner frees its slot."""
        if self._local == 0:
            return
        self._dist.barrier(group=self._group)   # every rank's kernels have finished (each rank synchronised before)
        if self.handle is not None:
            self._ops.heap_destroy(self.handle)
            self.handle = None
        for p in self._opened:
            self._ops.close(p)
        self._opened = []
        self._dist.barrier(group=self._group)   # nobody maps this rank's slot any more
        self._ops.free(self._local)
        self._local = 0

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        if exc[0] is None:
            self.close()
        else:
            self._release()   # an error on this rank: release without waiting for peers that may never arrive
        return False
