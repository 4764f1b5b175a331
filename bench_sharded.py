"""A benchmark configuration run block-sharded over the ranks of one node
(harness for `bench.py --shard-blocks` and for the tests; the product side —
ownership map, peer buffers, interprocess events, the per-rank service — is
paper_2204_03211_b200/sharded.py).

Rank r owns the blocks `sharded.partition` gives it and, as a worker host, holds
the gradient shards of the workers w with w mod world == r of EVERY job in one
exported buffer: job after job, worker after worker, each shard row padded to
128 elements.  Every rank can compute every rank's layout, so only 64-byte
handles travel.

Two transports for a block's W shards:
  inplace  the owner maps the workers' buffers and its aggregation kernel reads
           the shards where they are (over NVLink when the GPUs differ);
  staged   the worker's process copies its shard into a staging buffer that the
           OWNER exports (plain copies by the copy engines, issued ahead of the
           aggregate), so the pushes arrive in the owner's own memory and its
           kernel reads local HBM only; the owner's stream waits for the copies
           through interprocess events, no host waits for a device.

A block changes owner by a migration between services (the paper's Section 3.2
and Appendix B): export into a lane buffer, import on the new owner, ordered by
interprocess events; the old owner forgets the block at the next step.
"""
from __future__ import annotations

import numpy as np
import torch

from paper_2204_03211_b200 import binding as B
from paper_2204_03211_b200.sharded import (PeerEvents, PeerSlabs, ShardedService, device_bytes, partition,
                                           worker_rank)
from workload import configs, generate


class ShardedWorkload:
    """`exchange(obj) -> list` is an all-gather of a picklable object over the
    ranks; `barrier()` blocks until every rank has called it."""

    ROW_ALIGN = 128

    def __init__(self, cfg, rank: int, world: int, device: int, exchange, barrier, arena_slack: int = 64 << 20,
                 param_device="cpu", transport: str = "inplace", lane_bytes: int = 0):
        assert transport in ("inplace", "staged")
        self.cfg, self.rank, self.world, self.device = cfg, rank, world, device
        self.barrier, self.exchange, self.transport = barrier, exchange, transport
        costs = {(j, b.block): job.bytes_per_elem() * b.nelem for j, job in enumerate(cfg.jobs) for b in job.blocks}
        owner = partition(costs, world)
        mine = [(j, b) for j, job in enumerate(cfg.jobs) for b in job.blocks if owner[(j, b.block)] == rank]
        arena = sum(3 * (4 * b.nelem + 256) for _, b in mine) + arena_slack
        self.sh = ShardedService(rank, world, device, cfg.num_contexts, arena)
        self.sh.set_owners(owner)
        self._account()
        # layout of every rank's exported gradient buffer
        self.row_off = {}                       # (job, worker) -> byte offset inside its host rank's buffer
        size = [0] * world
        for j, job in enumerate(cfg.jobs):
            esz = self._esz(j)
            row = (job.num_params + self.ROW_ALIGN - 1) // self.ROW_ALIGN * self.ROW_ALIGN * esz
            for w in range(job.num_workers):
                r = worker_rank(w, world)
                self.row_off[(j, w)] = size[r]
                size[r] += row
        self.slabs = PeerSlabs(rank, world, device, size[rank], exchange)
        # staged transport: every owner exports room for the shards of its blocks that come from OTHER ranks
        self.stage_off, self.staging, self.staged_ev = {}, None, None
        self.nvlink_bytes_per_step = 0          # bytes this rank's workers send to other ranks per step
        if transport == "staged":
            # per owner: job after job, worker after worker, that worker's shards of the owner's blocks in block
            # order, each at the same position inside a 256-byte line as its source (same alignment class, and
            # consecutive blocks of one owner stay adjacent, so they travel as one copy)
            ssize = [0] * world
            for j, job in enumerate(cfg.jobs):
                for w in range(job.num_workers):
                    for b in job.blocks:
                        o = owner[(j, b.block)]
                        if worker_rank(w, world) == o:
                            continue            # already in the owner's memory
                        n = b.nelem * self._esz(j)
                        src_mod = (self.row_off[(j, w)] + b.job_offset * self._esz(j)) % 256
                        off = ssize[o] + (src_mod - ssize[o]) % 256
                        self.stage_off[(j, b.block, w)] = off
                        ssize[o] = off + n
                        if worker_rank(w, world) == rank:
                            self.nvlink_bytes_per_step += n
            self.staging = PeerSlabs(rank, world, device, max(ssize[rank], 256), exchange)
            self.staged_ev = PeerEvents(rank, world, device, exchange)
            self._stage_lists = None
        else:
            # in place: what this rank's kernels read from other ranks' memory per step
            for (j, blk), o in owner.items():
                if o != rank:
                    continue
                job = cfg.jobs[j]
                self.nvlink_bytes_per_step += sum(job.blocks[blk].nelem * self._esz(j) for w in range(job.num_workers)
                                                  if worker_rank(w, world) != rank)
        # migration between services: one lane buffer per rank (allocated once), two events per rank
        need = lane_bytes or max([self.packed_bytes(j, b.block) for j, b in mine] + [256]) * 8
        self.lane = PeerSlabs(rank, world, device, need, exchange)
        self.lane_bytes = exchange(need)
        self.exported_ev = PeerEvents(rank, world, device, exchange)
        self.imported_ev = PeerEvents(rank, world, device, exchange)
        self._imports_pending = False           # peers may still be reading this rank's lane
        self._retired = []                      # blocks this rank gave away and has not unregistered yet
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

    # ------------------------------------------------------------------ layout

    def _esz(self, job: int) -> int:
        return 2 if self.cfg.jobs[job].grad_dtype == configs.BF16 else 4

    def _account(self):
        own = [(j, b) for (j, b), r in self.sh.owner.items() if r == self.rank]
        self.owned_params = sum(self.cfg.jobs[j].blocks[b].nelem for j, b in own)
        self.owned_bytes = sum(self.cfg.jobs[j].bytes_per_elem() * self.cfg.jobs[j].blocks[b].nelem for j, b in own)

    def close(self):
        torch.cuda.synchronize(self.device)
        self.barrier()                          # nobody reads a peer's buffer any more
        self._retire()
        self.close_arenas()
        for ev in (self.staged_ev, self.exported_ev, self.imported_ev):
            if ev is not None:
                ev.close()
        self.barrier()                          # every mapping of an arena is gone before its service goes
        for slabs in (self.staging, self.lane, self.slabs):
            if slabs is not None:
                slabs.close(self.barrier)
        self.sh.close()

    def source_address(self, job: int, block: int, worker: int) -> int:
        """Address, in this process, of worker w's shard of (job, block) where the worker wrote it."""
        spec = self.cfg.jobs[job]
        return (self.slabs.base[worker_rank(worker, self.world)] + self.row_off[(job, worker)]
                + spec.blocks[block].job_offset * self._esz(job))

    def shard_address(self, job: int, block: int, worker: int) -> int:
        """Address the OWNER pushes for worker w's shard of (job, block): the
        worker's buffer (in place), or this rank's staging buffer (staged, for a
        shard that comes from another rank)."""
        if self.transport == "staged" and (job, block, worker) in self.stage_off \
                and self.sh.owner[(job, block)] == self.rank:
            return self.staging.own + self.stage_off[(job, block, worker)]
        return self.source_address(job, block, worker)

    def fill(self, iteration: int, gen_device="cpu"):
        """Writes this rank's workers' gradients of `iteration` into its exported
        buffer (the seeded generator's values, identical to the unsharded run
        that generates on the same kind of device), then meets the other ranks:
        on return every rank's buffer is complete."""
        dev = torch.device("cuda", self.device)
        for j, job in enumerate(self.cfg.jobs):
            slab = generate.grad_slab(self.cfg, j, iteration, gen_device)
            rowbytes = job.num_params * slab.element_size()
            for w in range(job.num_workers):
                if worker_rank(w, self.world) != self.rank:
                    continue
                dst = device_bytes(self.slabs.own + self.row_off[(j, w)], rowbytes, self.device)
                dst.copy_(slab[w].contiguous().view(torch.uint8).to(dev))      # no-op move when generated on dev
            del slab
        torch.cuda.synchronize(dev)
        self.barrier()

    # ------------------------------------------------------------------ staged transport

    def stage(self, stream=None):
        """Staged transport, the workers' half of a step: copies this rank's
        workers' shards of blocks owned elsewhere into the owners' staging buffers
        (runs of consecutive blocks with one owner travel as one copy), then
        records this rank's event.  Returns the bytes sent."""
        if self._stage_lists is None:
            runs = []
            for j, job in enumerate(self.cfg.jobs):
                for w in range(job.num_workers):
                    if worker_rank(w, self.world) != self.rank:
                        continue
                    run = None                  # [dst, src, bytes] of the run being extended
                    for b in job.blocks:
                        o = self.sh.owner[(j, b.block)]
                        n = b.nelem * self._esz(j)
                        if o == self.rank:
                            run = None
                            continue
                        dst = self.staging.base[o] + self.stage_off[(j, b.block, w)]
                        src = self.source_address(j, b.block, w)
                        if run is not None and run[0] + run[2] == dst and run[1] + run[2] == src:
                            run[2] += n
                        else:
                            run = [dst, src, n]
                            runs.append(run)       # extended in place while the next blocks are adjacent
            self._stage_lists = (np.array([r[0] for r in runs], np.uint64), np.array([r[1] for r in runs], np.uint64),
                                 np.array([r[2] for r in runs], np.uint64))
        d, s_, n = self._stage_lists
        if len(d):
            B.ps_peer_copy_many(d, s_, n, stream)
        self.staged_ev.record(stream)
        return int(n.sum()) if len(n) else 0

    def wait_staged(self, stream=None):
        """The owners' half: this rank's stream waits for every other rank's
        copies.  Call it after a host exchange that follows every rank's stage()."""
        for r in range(self.world):
            if r != self.rank:
                self.staged_ev.wait(r, stream)

    # ------------------------------------------------------------------ pull across ranks

    def open_arenas(self, exchange=None):
        """Collective: every rank exports the arenas of its service and tells where
        its blocks live; afterwards `param_address` works for every block.  Call
        again after a migration (locations change)."""
        exchange = exchange or self.exchange
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

    # ------------------------------------------------------------------ migration between services

    def packed_bytes(self, job: int, block: int) -> int:
        """Size of a block's packed state (parameters and optimizer state, each
        section rounded up to 256 bytes): what a migration moves."""
        spec = self.cfg.jobs[job]
        sec = (4 * spec.blocks[block].nelem + 255) // 256 * 256
        return sec * (3 if spec.opt == 1 else 2)

    def _retire(self):
        """Forgets the blocks this rank has given away (waits, on the host, only
        for its own export copies of them, which have long finished by now)."""
        for (j, b) in self._retired:
            self.sh.svc.unregister_block(j, b)
        self._retired = []

    def migrate(self, moves, exchange=None, stream=None):
        """Changes the owner of blocks: moves = [(job, block, new_rank)], the
        same list on every rank (a collective call, like a migration ordered by
        the paper's pMaster).  No host waits for its device: the old owner
        enqueues the copies of the blocks' packed state into its lane buffer and
        records its `exported` event; after a host exchange (which only says
        "the record call has been made") the new owner registers the blocks,
        makes its stream wait for that event and enqueues the imports — later
        aggregates of those blocks wait for the import by the library's own
        event — and records `imported`, which the old owner's next export waits
        for before it overwrites the lane.  The old owner forgets the blocks at
        its next step.  The new owner's arena must have room for the block
        (`arena_slack` at construction).  Returns the bytes this rank sent."""
        exchange = exchange or self.exchange
        if self.transport == "staged":
            raise NotImplementedError("owner changes under the staged transport need the staging layout rebuilt")
        self._retire()
        moves = [(j, b, r) for (j, b, r) in moves if self.sh.owner[(j, b)] != r]
        out = [(j, b, r) for (j, b, r) in moves if self.sh.owner[(j, b)] == self.rank]
        offs, off_by_rank = {}, [0] * self.world
        for (j, b, r) in moves:                        # every rank derives every offset
            src = self.sh.owner[(j, b)]
            offs[(j, b)] = off_by_rank[src]
            off_by_rank[src] += self.packed_bytes(j, b)
        for r in range(self.world):
            if off_by_rank[r] > self.lane_bytes[r]:
                raise ValueError("rank %d would export %d bytes through a lane of %d: move fewer blocks per call "
                                 "or construct with a larger lane_bytes" % (r, off_by_rank[r], self.lane_bytes[r]))
        # host-only: the step counters travel with the first exchange, which also tells every rank that all the
        # others have left their previous migrate() (so their `imported` records have been issued)
        steps = {(j, b): self.sh.svc.block_export(j, b)[1] for (j, b, _) in out}
        all_steps = {}
        for d in exchange(steps):
            all_steps.update(d)
        if out:
            if self._imports_pending:
                for r in range(self.world):
                    if r != self.rank:
                        self.imported_ev.wait(r, stream)   # the lane's previous readers are done before it is rewritten
            for (j, b, r) in out:
                n = self.packed_bytes(j, b)
                got, _ = self.sh.svc.block_export(j, b, self.lane.own + offs[(j, b)], n, stream)
                assert got == n
        self.exported_ev.record(stream)
        exchange(len(out))                             # "my record call has been made": no device is waited for
        sources = sorted({self.sh.owner[(j, b)] for (j, b, r) in moves if r == self.rank})
        for src in sources:
            self.exported_ev.wait(src, stream)
        for (j, b, r) in moves:
            if r != self.rank:
                continue
            src = self.sh.owner[(j, b)]
            spec = self.cfg.jobs[j]
            self.sh.svc.register_block(j, b, spec.blocks[b].nelem, 0, None)
            self.sh.svc.block_import(j, b, self.lane.base[src] + offs[(j, b)], self.packed_bytes(j, b),
                                     all_steps[(j, b)], stream)
        self.imported_ev.record(stream)
        self._imports_pending = True
        self._retired += [(j, b) for (j, b, r) in out]
        for (j, b, r) in moves:
            self.sh.owner[(j, b)] = r
        self._args.clear()
        self._account()
        return sum(self.packed_bytes(j, b) for (j, b, _) in out)

    # ------------------------------------------------------------------ steps

    def _round_args(self, key, ready):
        if key not in self._args:
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
        """Push and aggregate this rank's blocks of every round; returns the
        number of rounds it had work in.  `key` names the schedule so that call
        arguments are built once.  The launches are ordered after the work
        enqueued on `stream` (under the staged transport: after wait_staged)."""
        self._retire()
        n = 0
        for i, ready in enumerate(rounds):
            mine, jobs, blocks, workers, ptrs, tasks = self._round_args((key, i), ready)
            if not mine:
                continue
            self.sh.svc.round(jobs, blocks, workers, ptrs, tasks, 0, stream)
            n += 1
        return n
