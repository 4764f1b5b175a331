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

A block changes owner by a migration between services (`ShardedWorkload.migrate`:
ps_block_export into an exported buffer, ps_block_import on the new owner,
ps_unregister_block on the old one).

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


class ShardedWorkload:
    """A benchmark configuration (workload.configs.Config) run block-sharded.

    Rank r owns the blocks `partition` gives it and, as a worker host, holds the
    gradient shards of workers w with w mod world == r of EVERY job in one
    exported buffer: job after job, worker after worker, each shard row padded
    to 128 elements.  Every rank can compute every rank's layout, so only the
    64-byte handles travel.  `exchange` as in PeerSlabs; `barrier()` blocks
    until every rank has called it."""

    ROW_ALIGN = 128

    def __init__(self, cfg, rank: int, world: int, device: int, exchange, barrier, arena_slack: int = 64 << 20,
                 param_device="cpu"):
        import numpy as np
        from workload import configs, generate
        self.cfg, self.rank, self.world, self.device = cfg, rank, world, device
        self.barrier = barrier
        self._generate, self._np = generate, np
        costs = {(j, b.block): job.bytes_per_elem() * b.nelem for j, job in enumerate(cfg.jobs) for b in job.blocks}
        owner = partition(costs, world)
        mine = [(j, b) for j, job in enumerate(cfg.jobs) for b in job.blocks if owner[(j, b.block)] == rank]
        arena = sum(3 * (4 * b.nelem + 256) for _, b in mine) + arena_slack
        self.sh = ShardedService(rank, world, device, cfg.num_contexts, arena)
        self.sh.set_owners(owner)
        self.owned_params = sum(b.nelem for _, b in mine)
        self.owned_bytes = sum(costs[(j, b.block)] for j, b in mine)
        # layout of every rank's exported buffer
        self.row_off = {}                       # (job, worker) -> byte offset inside its host rank's buffer
        size = [0] * world
        for j, job in enumerate(cfg.jobs):
            esz = 2 if job.grad_dtype == configs.BF16 else 4
            row = (job.num_params + self.ROW_ALIGN - 1) // self.ROW_ALIGN * self.ROW_ALIGN * esz
            for w in range(job.num_workers):
                r = worker_rank(w, world)
                self.row_off[(j, w)] = size[r]
                size[r] += row
        self.slabs = PeerSlabs(rank, world, device, size[rank], exchange)
        self._arena_base = None
        for j, job in enumerate(cfg.jobs):
            assert self.sh.register_job(**job.hparams()) == j
            p0 = generate.init_params(cfg, j, param_device)     # the seeded generator of that device kind
            for b in job.blocks:
                if owner[(j, b.block)] == rank:
                    self.sh.register_block(j, b.block, b.nelem, configs.initial_context(cfg, j, b.block),
                                           p0[b.job_offset:b.job_offset + b.nelem].contiguous())
            del p0
        self._args = {}

    def close(self):
        import torch
        torch.cuda.synchronize(self.device)
        self.barrier()                          # nobody reads a peer's buffer any more
        self.close_arenas()
        self.barrier()                          # every mapping of an arena is gone before its service goes
        self.slabs.close(self.barrier)
        self.sh.close()

    def shard_address(self, job: int, block: int, worker: int) -> int:
        """Address, in this process, of worker w's shard of (job, block)."""
        spec = self.cfg.jobs[job]
        esz = 2 if spec.grad_dtype == 1 else 4
        return (self.slabs.base[worker_rank(worker, self.world)] + self.row_off[(job, worker)]
                + spec.blocks[block].job_offset * esz)

    def fill(self, iteration: int, gen_device="cpu"):
        """Writes this rank's workers' gradients of `iteration` into its exported
        buffer (the seeded generator's values, identical to the unsharded run
        that generates on the same kind of device), then meets the other ranks:
        on return every rank's buffer is complete."""
        import torch
        dev = torch.device("cuda", self.device)
        for j, job in enumerate(self.cfg.jobs):
            slab = self._generate.grad_slab(self.cfg, j, iteration, gen_device)
            rowbytes = job.num_params * slab.element_size()
            for w in range(job.num_workers):
                if worker_rank(w, self.world) != self.rank:
                    continue
                dst = device_bytes(self.slabs.own + self.row_off[(j, w)], rowbytes, self.device)
                dst.copy_(slab[w].contiguous().view(torch.uint8).to(dev))      # no-op move when generated on dev
            del slab
        torch.cuda.synchronize(dev)
        self.barrier()

    def open_arenas(self, exchange):
        """Collective: every rank exports the arenas of its service and tells where
        its blocks live; afterwards `param_address` works for every block.  Call
        again after a migration (locations change)."""
        self.close_arenas()
        nctx = self.cfg.num_contexts
        mine = [self.sh.svc.arena_export(c)[0] for c in range(nctx)]
        where = {k: self.sh.svc.block_location(*k)[:2] for k, r in self.sh.owner.items() if r == self.rank}
        self._arena_base, self._where = [None] * self.world, {}
        for r, (handles, loc) in enumerate(exchange((mine, where))):
            self._where.update(loc)
            if r != self.rank:
                self._arena_base[r] = [B.ps_peer_open(self.device, h) for h in handles]

    def close_arenas(self):
        for bases in getattr(self, "_arena_base", None) or []:
            for p in bases or []:
                B.ps_peer_close(self.device, p)
        self._arena_base = None

    def param_address(self, job: int, block: int) -> int:
        """Pull from anywhere: address, in this process, of the block's nelem fp32
        parameters — in the local arena or in the owner's mapped one."""
        r = self.sh.owner[(job, block)]
        if r == self.rank:
            return self.sh.pull(job, block)
        ctx, off = self._where[(job, block)]
        return self._arena_base[r][ctx] + off

    def packed_bytes(self, job: int, block: int) -> int:
        """Size of a block's packed state (parameters and optimizer state, each
        section rounded up to 256 bytes): what a migration moves."""
        spec = self.cfg.jobs[job]
        sec = (4 * spec.blocks[block].nelem + 255) // 256 * 256
        return sec * (3 if spec.opt == 1 else 2)

    def migrate(self, moves, exchange, stream=None):
        """Changes the owner of blocks: moves = [(job, block, new_rank)], the
        same list on every rank (a collective call, like a migration ordered by
        the paper's pMaster).  The old owner copies the block's packed state into
        a buffer it exports, the new owner registers the block and copies it in
        from its mapping of that buffer, then the old owner forgets the block.
        Aggregates of a moved block that the new owner enqueues afterwards wait
        for the copy.  The new owner's arena must have room for the block
        (`arena_slack` at construction) before the old owner releases its range.
        Returns the bytes this rank sent."""
        import torch
        moves = [(j, b, r) for (j, b, r) in moves if self.sh.owner[(j, b)] != r]
        out = [(j, b, r) for (j, b, r) in moves if self.sh.owner[(j, b)] == self.rank]
        size = sum(self.packed_bytes(j, b) for j, b, _ in out)
        lane = PeerSlabs(self.rank, self.world, self.device, size, exchange)
        offs, off_by_rank = {}, [0] * self.world
        for (j, b, r) in moves:                        # every rank derives every offset
            src = self.sh.owner[(j, b)]
            offs[(j, b)] = off_by_rank[src]
            off_by_rank[src] += self.packed_bytes(j, b)
        steps = {}
        for (j, b, r) in out:
            n = self.packed_bytes(j, b)
            got, step = self.sh.svc.block_export(j, b, lane.own + offs[(j, b)], n, stream)
            assert got == n
            steps[(j, b)] = step
        torch.cuda.synchronize(self.device)            # the exported copies have landed ...
        all_steps = {}
        for d in exchange(steps):                      # ... and this exchange is the barrier that says so
            all_steps.update(d)
        for (j, b, r) in moves:
            if r != self.rank:
                continue
            src = self.sh.owner[(j, b)]
            spec = self.cfg.jobs[j]
            self.sh.owner[(j, b)] = r
            self.sh.svc.register_block(j, b, spec.blocks[b].nelem, 0, None)
            self.sh.svc.block_import(j, b, lane.base[src] + offs[(j, b)], self.packed_bytes(j, b),
                                     all_steps[(j, b)], stream)
        torch.cuda.synchronize(self.device)            # the imports have read the lanes
        self.barrier()
        for (j, b, r) in out:
            self.sh.svc.unregister_block(j, b)
        for (j, b, r) in moves:
            self.sh.owner[(j, b)] = r
        lane.close(self.barrier)
        self._args.clear()
        self.owned_params = sum(self.cfg.jobs[j].blocks[b].nelem for (j, b), r in self.sh.owner.items() if r == self.rank)
        self.owned_bytes = sum(self.cfg.jobs[j].bytes_per_elem() * self.cfg.jobs[j].blocks[b].nelem
                               for (j, b), r in self.sh.owner.items() if r == self.rank)
        return size

    def _round_args(self, key, ready):
        if key not in self._args:
            np = self._np
            mine = self.sh.owned(ready)
            jobs, blocks, workers, ptrs = [], [], [], []
            for (j, b) in mine:
                for w in range(self.cfg.jobs[j].num_workers):
                    jobs.append(j); blocks.append(b); workers.append(w)
                    ptrs.append(self.shard_address(j, b, w))
            self._args[key] = (mine, np.array(jobs, np.int32), np.array(blocks, np.int32),
                               np.array(workers, np.int32), np.array(ptrs, np.uint64), B.make_tasks(mine))
        return self._args[key]

    def step(self, rounds, stream=None, key=0) -> int:
        """Push and aggregate this rank's blocks of every round; returns launches.
        `key` names the schedule so that call arguments are built once."""
        launches = 0
        for i, ready in enumerate(rounds):
            mine, jobs, blocks, workers, ptrs, tasks = self._round_args((key, i), ready)
            if not mine:
                continue
            self.sh.svc.push_batch(jobs, blocks, workers, ptrs)
            self.sh.svc.aggregate(tasks, stream)
            launches += 1
        return launches
