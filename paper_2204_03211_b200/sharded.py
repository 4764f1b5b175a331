"""Block-sharded deployment: several Aggregators on the GPUs of one node.

The paper spreads the tensors of a job over several Aggregators, which exchange
nothing with one another except migrated tensors (Section 3.2; aggregation
tasks are independent per tensor, Section 2.2).  Here one process per GPU runs
one service; every (job, block) has ONE owner rank, which holds its master copy
and runs its aggregation.  There is no collective in the aggregation path: the
W gradient shards of a block sit in buffers that the workers' processes export
(`ps_peer_alloc`), the owner maps them (`ps_peer_open`) and pushes the mapped
addresses, and the aggregation kernel reads them in place — through NVLink when
the worker's GPU is not the owner's.

A block changes owner by a migration between services: ps_block_export into an
exported buffer, ps_block_import on the new owner, ps_unregister_block on the
old one, ordered by interprocess events (`PeerEvents`) so that neither host
waits for its device.

This module is host logic only (who owns what, which address a shard has in
which process); every arithmetic step runs in the library's kernels.
"""
from __future__ import annotations

from . import binding as B


def partition(costs: dict, world: int) -> dict:
    """Owner rank of every key of `costs` ({(job, block): cost}, cost = bytes the
    block's aggregation moves).  Longest-processing-time greedy: heaviest block
    first, to the least-loaded rank, lowest rank on ties; keys break cost ties.
    Deterministic, so every rank computes the same map without communicating.
    The heaviest rank carries at most 4/3 of the optimum (Graham's bound)."""
    if world < 1:
        raise ValueError("world must be >= 1")
    load = [0.0] * world
    owner = {}
    for key in sorted(costs, key=lambda k: (-costs[k], k)):
        r = min(range(world), key=lambda i: (load[i], i))
        owner[key] = r
        load[r] += costs[key]
    return owner


def worker_rank(worker: int, world: int) -> int:
    """Rank whose process holds worker w's shards (workers dealt round-robin)."""
    return worker % world


class PeerSlabs:
    """One exported device buffer per rank, mapped by every other rank.

    `exchange(obj) -> list` is an all-gather of a picklable object over the
    ranks (e.g. `torch.distributed.all_gather_object`).  `base[r]` is the
    address of rank r's buffer in THIS process (its own buffer: the pointer
    itself).  A rank that needs no buffer passes nbytes = 0."""

    def __init__(self, rank: int, world: int, device: int, nbytes: int, exchange):
        self.rank, self.world, self.device = rank, world, device
        self.own, handle = (B.ps_peer_alloc(device, nbytes) if nbytes > 0 else (0, b""))
        self.nbytes = nbytes
        handles = exchange(handle)
        if len(handles) != world:
            raise ValueError("exchange returned %d handles for %d ranks" % (len(handles), world))
        self.base, self._opened = [0] * world, []
        for r, h in enumerate(handles):
            if r == rank:
                self.base[r] = self.own
            elif h:
                self.base[r] = B.ps_peer_open(device, h)
                self._opened.append(self.base[r])

    def close(self, barrier=None):
        """Unmaps the peers' buffers and frees this rank's own.  Call it on every
        rank only after all ranks have finished using the buffers.  With
        `barrier` (a callable every rank calls) no rank frees its buffer before
        every rank has unmapped it."""
        for p in self._opened:
            B.ps_peer_close(self.device, p)
        self._opened = []
        if barrier is not None:
            barrier()
        if self.own:
            B.ps_peer_free(self.device, self.own)
            self.own = 0


class ShardedService:
    """The local service of one rank plus the ownership map.

    Jobs are registered on every rank in the same order (hyper-parameters are a
    few bytes); a block is registered only in its owner's service.  push /
    aggregate / pull act on owned blocks and ignore the others, so every rank can
    run the same loop over the whole ready list."""

    def __init__(self, rank: int, world: int, device: int, num_contexts: int = 1, arena_bytes: int = 1 << 30):
        self.rank, self.world, self.device = rank, world, device
        self.svc = B.Service(device, num_contexts, arena_bytes)
        self.owner = {}

    def close(self):
        self.svc.close()

    def register_job(self, **hp) -> int:
        return self.svc.register_job(**hp)

    def set_owners(self, owner: dict):
        self.owner = dict(owner)

    def owns(self, job: int, block: int) -> bool:
        return self.owner[(job, block)] == self.rank

    def register_block(self, job: int, block: int, nelem: int, ctx: int = 0, init=None) -> bool:
        if not self.owns(job, block):
            return False
        self.svc.register_block(job, block, nelem, ctx, init)
        return True

    def push(self, job: int, block: int, worker: int, ptr) -> bool:
        """`ptr`: the shard's address in THIS process (a mapped peer address or a
        local one)."""
        if not self.owns(job, block):
            return False
        self.svc.push(job, block, worker, ptr)
        return True

    def owned(self, ready) -> list:
        return [(j, b) for (j, b) in ready if self.owns(j, b)]

    def aggregate(self, ready, stream=None) -> int:
        """One packed launch for the owned tasks of `ready`; returns how many."""
        mine = self.owned(ready)
        if mine:
            self.svc.aggregate(mine, stream)
        return len(mine)

    def pull(self, job: int, block: int) -> int:
        if not self.owns(job, block):
            raise B.PsError(B.PS_ERR_BAD_ARG, "ShardedService.pull", "block (%d,%d) is owned by rank %d" % (
                job, block, self.owner[(job, block)]))
        return self.svc.pull(job, block)


def device_bytes(ptr: int, nbytes: int, device: int):
    """uint8 torch view of device memory that torch did not allocate (no copy)."""
    import torch

    class _Mem:
        pass

    m = _Mem()
    m.__cuda_array_interface__ = {"shape": (nbytes,), "typestr": "|u1", "data": (ptr, False), "version": 2}
    return torch.as_tensor(m, device="cuda:%d" % device)


class PeerEvents:
    """One interprocess event per rank, opened by every other rank.

    `mine` is recorded by this rank on one of its streams; `wait(r, stream)`
    makes a local stream wait for rank r's most recent record.  The record call
    must have been issued before the wait is enqueued: the ranks tell each other
    so over their host channel (any exchange after the record will do); nobody
    waits for a device.  `exchange` as in PeerSlabs."""

    def __init__(self, rank: int, world: int, device: int, exchange):
        self.rank, self.world, self.device = rank, world, device
        self.mine, handle = B.ps_peer_event_create(device)
        self.events = [None] * world
        for r, h in enumerate(exchange(handle)):
            self.events[r] = self.mine if r == rank else B.ps_peer_event_open(device, h)

    def record(self, stream=None):
        B.ps_peer_event_record(self.mine, stream)

    def wait(self, r: int, stream=None):
        B.ps_peer_event_wait(self.events[r], stream)

    def close(self):
        for ev in self.events:
            if ev:
                B.ps_peer_event_destroy(ev)
        self.events = []
