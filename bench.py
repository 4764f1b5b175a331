#!/usr/bin/env python
"""Benchmark of the packed model-aggregation hot path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload C4]

A step is one BSP iteration of every job of the workload: each block receives
its W pushes, becomes ready in one of the rounds of the seeded arrival
schedule, is aggregated (one packed kernel launch per round) and pulled.
Default workload: the 12 packed concurrent jobs (661 M parameters, 31.03 GB of
algorithmic HBM traffic per step).  Prints ONE JSON line.

`value` is timed with gradients resident in HBM; `e2e` pushes from pinned host
memory and pulls parameters back to the host inside the timed region.
`--impl reference` times the CPU oracle on a bounded sample of the same
workload (it is the only reference this path has).
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from workload import configs, generate  # noqa: E402

METRIC = "aggregated_params_per_sec"
UNIT = "params/s"
FALLBACK_HBM_GBS = 6650.0

# DRAM traffic of the dominant kernel from the committed ncu captures
# (profiles/), as measured dram bytes per algorithmic byte, per kernel, keyed by
# the hash of the kernel source it was taken from.  A changed kernel (or one
# without a capture) reports null.
_SHARED_SOURCES = ("ps_types.cuh", "ps_math.cuh", "ps_rows.cuh")
NCU_TRAFFIC = {
    "ps_aggregate_ldg_kernel": {"sources": _SHARED_SOURCES + ("ps_kernel_ldg.cuh",), "kernel_sha": "4733ace9e33e",
                                "dram_bytes_per_algorithmic_byte": 0.980},
    "ps_aggregate_bulk_kernel": {"sources": _SHARED_SOURCES + ("ps_kernel_bulk.cuh",), "kernel_sha": "5610a06cdf42",
                                 "dram_bytes_per_algorithmic_byte": 0.984},
}


def kernel_sha(kernel: str = "ps_aggregate_ldg_kernel") -> str:
    h = hashlib.sha256()
    for name in NCU_TRAFFIC.get(kernel, NCU_TRAFFIC["ps_aggregate_ldg_kernel"])["sources"]:
        with open(os.path.join(ROOT, "paper_2204_03211_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:12]


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ------------------------------------------------------------------ clocks

class ClockSampler:
    """Samples nvidia-smi every 50 ms from before the warm-up until the timed
    region ends.  clocks.sm / clocks.max.sm are parsed on their own; the
    throttle-reason fields are optional (a driver that does not know one of
    them falls back to a query of the two clock fields only)."""
    FULL = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
            "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
            "clocks_event_reasons.sw_power_cap")
    BASIC = "clocks.sm,clocks.max.sm"
    REASONS = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.path, self.fields, self.note = index, None, None, self.FULL, None
        self.marks = []

    def _spawn(self, fields):
        fd, self.path = tempfile.mkstemp(suffix=".csv")
        os.close(fd)
        self.fields = fields
        self.proc = subprocess.Popen(
            ["nvidia-smi", "-i", str(self.index), "--query-gpu=timestamp," + fields,
             "--format=csv,noheader,nounits", "-lms", "50"],
            stdout=open(self.path, "w"), stderr=subprocess.STDOUT)

    def start(self):
        try:
            self._spawn(self.FULL)
            time.sleep(0.25)
            if self.proc.poll() is not None:           # refused the query: ask for the clocks alone
                self.note = "full query refused: " + open(self.path).read().strip()[:120]
                self._spawn(self.BASIC)
        except Exception as e:                         # noqa: BLE001
            self.proc, self.note = None, "nvidia-smi could not be started: %r" % (e,)

    def mark(self):
        """Remembers 'now' (the sampler's own clock: lines written so far)."""
        try:
            with open(self.path) as f:
                self.marks.append(sum(1 for _ in f))
        except Exception:
            self.marks.append(0)

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "samples_timed_region": 0}
        if not self.proc:
            out["why_no_samples"] = self.note or "sampler not started"
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        rows, bad = [], 0
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                try:
                    rows.append((float(f[1]), float(f[2]), f[3:]))
                except (ValueError, IndexError):
                    bad += 1
                    rows.append(None)
            os.unlink(self.path)
        except Exception as e:                         # noqa: BLE001
            out["why_no_samples"] = "cannot read the sampler's output: %r" % (e,)
            return out
        first = self.marks[0] if self.marks else 0
        timed = [r for r in rows[first:] if r]
        every = [r for r in rows if r]
        use = timed if timed else every
        if not use:
            out["why_no_samples"] = (self.note or "") + " no parsable line among %d (%d unparsable)" % (len(rows), bad)
            return out
        # under load = the upper half of the samples of the timed region (the lower half may hold the
        # gaps between blocks of steps)
        sm = sorted(r[0] for r in use)
        upper = sm[len(sm) // 2:]
        reasons = set()
        if self.fields == self.FULL:
            for r in use:
                for name, v in zip(self.REASONS, r[2][1:5]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
        out.update(sm_mhz=statistics.median(upper), sm_max_mhz=max(r[1] for r in use), reasons=sorted(reasons),
                   samples=len(every), samples_timed_region=len(timed), sm_mhz_min=sm[0])
        if self.note:
            out["note"] = self.note
        return out


# ------------------------------------------------------------------ our arm

class Workload:
    """The service, the device-resident gradients and the per-round call
    arguments of one workload, prepared outside any timed region."""

    def __init__(self, cfg: configs.Config, device: int, ticks: int, n_schedules: int, sparse: bool = False,
                 prepared: bool = True):
        from paper_2204_03211_b200 import binding as B
        self.B, self.cfg, self.device = B, cfg, device
        dev = torch.device("cuda", device)
        arena = sum(3 * (4 * b.nelem + 256) for j in cfg.jobs for b in j.blocks) + (64 << 20)
        self.svc = B.Service(device, cfg.num_contexts, arena)
        self.slabs = []
        for j, job in enumerate(cfg.jobs):
            assert self.svc.register_job(**job.hparams()) == j
            p0 = generate.init_params(cfg, j, dev)
            for b in job.blocks:
                self.svc.register_block(j, b.block, b.nelem, configs.initial_context(cfg, j, b.block),
                                        p0[b.job_offset:b.job_offset + b.nelem])
            del p0
            self.slabs.append(generate.grad_slab(cfg, j, 0, dev))
        torch.cuda.synchronize(dev)
        # row-sparse transport: blocks of embedding-like tensors are pushed as (row ids, packed rows)
        self.sparse = {}          # (job, block) -> [(ids, values, n_rows, row_len)] per worker
        self.sparse_saved = 0     # gradient bytes not read per step, net of the ids that are
        if sparse:
            for j, job in enumerate(cfg.jobs):
                for blk in job.blocks:
                    t = job.tensors[blk.tensor]
                    if not t.row_sparse:
                        continue
                    row_len = t.nelem // t.shape[0]
                    shards = generate.row_sparse_shards(self.slabs[j], blk.job_offset, blk.nelem, row_len)
                    self.sparse[(j, blk.block)] = [(i, v, int(i.numel()), row_len) for i, v in shards]
                    esz = self.slabs[j].element_size()
                    for i, v in shards:
                        self.sparse_saved += blk.nelem * esz - (v.numel() * esz + i.numel() * 4)
            torch.cuda.synchronize(dev)
        # call arguments per schedule (= arrival pattern of one iteration) and round
        self.schedules = []
        for it in range(n_schedules):
            rounds = []
            for ready in configs.rounds_for(cfg, it, ticks):
                jobs, blocks, workers, ptrs = [], [], [], []
                rows = []
                for (j, b) in ready:
                    job = cfg.jobs[j]
                    blk = job.blocks[b]
                    if (j, b) in self.sparse:
                        for w, (i, v, n, rl) in enumerate(self.sparse[(j, b)]):
                            rows.append((j, b, w, i.data_ptr(), n, rl, v.data_ptr()))
                        continue
                    for w in range(job.num_workers):
                        jobs.append(j); blocks.append(b); workers.append(w)
                        ptrs.append(generate.shard_ptr(self.slabs[j], w, blk.job_offset))
                rounds.append(dict(ready=ready, tasks=B.make_tasks(ready), pulled=np.empty(len(ready), np.uint64),
                                   rows=None if not rows else tuple(
                                       np.array([a[k] for a in rows], np.uint64 if k in (3, 6) else np.int32)
                                       for k in range(7)),
                                   jobs=np.array(jobs, np.int32), blocks=np.array(blocks, np.int32),
                                   workers=np.array(workers, np.int32), ptrs=np.array(ptrs, np.uint64)))
            for r in rounds:
                r["n"] = len(r["ready"])
                r["c_push"] = (len(r["jobs"]), r["jobs"].ctypes.data, r["blocks"].ctypes.data,
                               r["workers"].ctypes.data, r["ptrs"].ctypes.data)
                r["c_pulled"] = r["pulled"].ctypes.data
                r["c_round"] = r["c_push"] + (r["tasks"], r["n"])
                if r["rows"] is not None:
                    r["c_rows"] = (len(r["rows"][0]),) + tuple(a.ctypes.data for a in r["rows"])
            self.schedules.append(rounds)
        self.lib = B.load()
        self.overlap = False
        # the gradient slabs are written once, before any timed region: every push is of a
        # buffer that is already complete in memory
        self.round_flags = B.PS_ROUND_INPUTS_COMPLETE
        # the rounds recur every len(schedules) steps with the same buffers: prepared once
        self.prepared = prepared
        for rounds in self.schedules:
            for r in rounds:
                r["rid"] = None
                if prepared and r["rows"] is None:
                    r["rid"] = self.svc.round_prepare(r["jobs"], r["blocks"], r["workers"], r["ptrs"], r["tasks"],
                                                      self.round_flags)
        self.params_per_step = cfg.num_params
        self.bytes_per_step = cfg.bytes_per_round() - self.sparse_saved

    def step(self, k: int, stream) -> int:
        """Push, aggregate, pull — device-resident gradients.  Returns the number of rounds."""
        # The C entry points are called with arguments marshalled once, outside
        # the timed region (array addresses as integers): one C-ABI call per round
        # (ps_round_run = push, aggregate, pull of a prepared round; ps_round with the
        # full argument lists otherwise), plus one for row-sparse pushes if any.
        lib, h, sp = self.lib, self.svc.handle, int(stream.cuda_stream)
        rounds = self.schedules[k % len(self.schedules)]
        flags = self.round_flags
        for r in rounds:
            rc = 0
            if r["rid"] is not None:
                rc = lib.ps_round_run(h, r["rid"], sp, r["c_pulled"])
            else:
                if r["rows"] is not None:
                    rc = lib.ps_push_rows_batch(h, *r["c_rows"])
                if rc == 0:
                    rc = lib.ps_round(h, *r["c_round"], flags, sp, r["c_pulled"])
            if rc:
                raise self.B.PsError(rc, "bench step")
        if self.overlap:
            lib.ps_join(h, sp)      # the step's launches overlapped each other; the stream joins them here
        return len(rounds)

    # ---- end to end: host gradients in, host parameters out

    def prepare_host(self, pool_bytes: int):
        """Pinned host memory holding every worker's shard of every block in the
        layout ps_push_host_batch sends as few copies: job after job, block
        after block in id order, worker after worker, rows padded to 256 bytes.
        If the pool is smaller than the workload's gradients, later jobs reuse
        the pool from its start (the bytes that cross the link are the same)."""
        cfg = self.cfg
        job_bytes, row = [], {}
        for j, job in enumerate(cfg.jobs):
            esz = 2 if job.grad_dtype == configs.BF16 else 4
            tot = 0
            for b in job.blocks:
                row[(j, b.block)] = (b.nelem * esz + 255) // 256 * 256
                tot += row[(j, b.block)] * job.num_workers
            job_bytes.append(tot)
        total = sum(job_bytes)
        pool_bytes = max(min(pool_bytes, total), max(job_bytes))
        self.pool = torch.empty(pool_bytes, dtype=torch.uint8, pin_memory=True)
        # gradient bit patterns (device -> host copy of the slabs' first bytes, repeated)
        off = 0
        for sl in self.slabs:
            src = (sl._base if sl._base is not None else sl).view(-1).view(torch.uint8)
            n = min(src.numel(), pool_bytes - off)
            if n <= 0:
                break
            self.pool[off:off + n].copy_(src[:n])
            off += n
        while 0 < off < pool_bytes:
            n = min(off, pool_bytes - off)
            self.pool[off:off + n].copy_(self.pool[:n])
            off += n
        base, start, self.host_ptr = self.pool.data_ptr(), 0, {}
        for j, job in enumerate(cfg.jobs):
            if start + job_bytes[j] > pool_bytes:
                start = 0
            cur = start
            for b in job.blocks:
                for w in range(job.num_workers):
                    self.host_ptr[(j, b.block, w)] = base + cur
                    cur += row[(j, b.block)]
            start = cur
        self.out = torch.empty(cfg.num_params, dtype=torch.float32, pin_memory=True)
        self.pool_bytes = pool_bytes
        self.pull_stream = torch.cuda.Stream(torch.device("cuda", self.device))
        self.pull_done = torch.cuda.Event()
        self.h2d = sum(job.num_params * job.num_workers * (2 if job.grad_dtype == configs.BF16 else 4)
                       for job in cfg.jobs)
        self.d2h = cfg.num_params * 4
        self._out_off, acc = {}, 0
        for j, job in enumerate(cfg.jobs):
            self._out_off[j] = acc
            acc += job.num_params
        # call arguments per schedule and round: the host addresses of the round's shards
        self.host_args = []
        for rounds in self.schedules:
            per_round = []
            for r in rounds:
                ptrs = np.array([self.host_ptr[(int(j), int(b), int(w))]
                                 for j, b, w in zip(r["jobs"], r["blocks"], r["workers"])], np.uint64)
                outs = [(j, b, self.out.data_ptr() + 4 * (self._out_off[j] + cfg.jobs[j].blocks[b].job_offset))
                        for (j, b) in r["ready"]]
                per_round.append((ptrs, outs))
            self.host_args.append(per_round)

    def _pull_round(self, outs):
        # parameters travel back on a second stream (the library orders each copy after the
        # block's aggregate), so device-to-host traffic overlaps the next round's uploads
        svc, ps = self.svc, self.pull_stream
        for (j, b, dst) in outs:
            svc.pull_host(j, b, dst, ps)

    def _end_host_step(self, stream):
        self.pull_done.record(self.pull_stream)
        stream.wait_event(self.pull_done)           # the step ends when its last result is on the host
        if self.overlap:
            self.svc.join(stream)

    def step_host(self, k: int, stream) -> int:
        """End to end, staged: the round's shards are copied from pinned host
        memory into device staging (ps_push_host_batch: neighbours travel as one
        copy), aggregated, and the parameters copied back to the host."""
        svc = self.svc
        sched = k % len(self.schedules)
        rounds = self.schedules[sched]
        for r, (ptrs, outs) in zip(rounds, self.host_args[sched]):
            svc.push_host_batch(r["jobs"], r["blocks"], r["workers"], ptrs, stream)
            svc.aggregate(r["tasks"], stream)
            self._pull_round(outs)
        self._end_host_step(stream)
        return len(rounds)

    def step_host_mapped(self, k: int, stream) -> int:
        """End to end without staging copies: pinned host memory is addressable
        from the device, so the pinned shards are pushed as they are and the
        aggregation kernel reads them over PCIe in place; parameters return to
        the host as in step_host."""
        svc = self.svc
        sched = k % len(self.schedules)
        rounds = self.schedules[sched]
        for r, (ptrs, outs) in zip(rounds, self.host_args[sched]):
            svc.push_batch(r["jobs"], r["blocks"], r["workers"], ptrs)
            svc.aggregate(r["tasks"], stream)
            self._pull_round(outs)
        self._end_host_step(stream)
        return len(rounds)


def max_over_ranks(ms: float, device=None) -> float:
    """Slowest rank's time (every rank gets it).  No-op without a process group."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return ms
    t = torch.tensor([ms], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(units_per_rank_per_step: int, world: int, steps: int, ms: float) -> float:
    """Replicas only: every rank processes the same number of units; the job's
    throughput is all ranks' units over the slowest rank's time."""
    return world * units_per_rank_per_step * steps / (ms * 1e-3)


def timed(fn, steps: int, stream, dist_on: bool, device):
    """Times `steps` calls of fn(k, stream) with CUDA events on `stream`,
    bracketed by barrier + synchronize; returns (ms max over ranks, rounds, host ms)."""
    import torch.distributed as dist
    torch.cuda.synchronize(device)
    if dist_on:
        dist.barrier()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    rounds = 0
    host0 = time.perf_counter()
    with torch.cuda.stream(stream):
        t0.record(stream)
        for k in range(steps):
            rounds += fn(k, stream)
        t1.record(stream)
    host_ms = (time.perf_counter() - host0) * 1e3
    torch.cuda.synchronize(device)
    if dist_on:
        dist.barrier()
    ms = max_over_ranks(t0.elapsed_time(t1), device)
    return ms, rounds, host_ms


def timed_blocks(fn, steps: int, stream, dist_on: bool, device, min_seconds: float, max_blocks: int):
    """The timed region: blocks of exactly `steps` steps, each bracketed as in
    timed(), repeated until `min_seconds` of device time have been measured
    (every rank repeats the same number of times: the count is derived from
    the first block's max-over-ranks time).  Returns the blocks' times (ms),
    rounds and host ms."""
    ms, rounds, host = timed(fn, steps, stream, dist_on, device)
    blocks, n_rounds, host_ms = [ms], rounds, [host]
    want = int(min(max_blocks, max(1, -(-min_seconds * 1e3 // max(ms, 1e-3)))))
    for i in range(1, want):
        base = i * steps
        ms, rounds, host = timed(lambda k, st: fn(base + k, st), steps, stream, dist_on, device)
        blocks.append(ms)
        host_ms.append(host)
        n_rounds += rounds
    return blocks, n_rounds, host_ms


# ------------------------------------------------------------------ CPU oracle arm

def oracle_sample(cfg: configs.Config, slabs=None, max_bytes: float = 9e9):
    """Bounded sample of the workload for the CPU oracle: whole jobs, one of
    each model where the workload has several, until the byte budget is used.
    Returns (items for oracle.run_blocks, params, description)."""
    from oracle import aggregator as A
    picked, seen_models, budget = [], set(), 0
    for j, job in enumerate(cfg.jobs):
        cost = job.bytes_per_elem() * job.num_params
        if job.model in seen_models or budget + cost > max_bytes:
            continue
        seen_models.add(job.model)
        picked.append(j)
        budget += cost
    if not picked:      # a single job larger than the budget: take its first blocks
        picked = [0]
    items, params = [], 0
    for j in picked:
        job = cfg.jobs[j]
        hp = A.HParams(**job.hparams())
        if slabs is not None:
            host = slabs[j].cpu()
        else:
            host = generate.grad_slab(cfg, j, 0)
        host = host.view(torch.int16).numpy().view(np.uint16) if host.dtype == torch.bfloat16 else host.numpy()
        p0 = generate.init_params(cfg, j).numpy()
        used = 0
        for b in job.blocks:
            if len(picked) == 1 and used * job.bytes_per_elem() > max_bytes:
                break
            sl = slice(b.job_offset, b.job_offset + b.nelem)
            p = p0[sl].copy()
            s0 = np.zeros(b.nelem, np.float32)
            s1 = np.zeros(b.nelem, np.float32) if job.opt == configs.ADAM else None
            items.append((hp, 1, [host[w, sl] for w in range(job.num_workers)], p, s0, s1))
            used += b.nelem
        params += used
    desc = "one aggregate of jobs %s of %s (%d blocks, %d params)" % (
        [cfg.jobs[j].name for j in picked], cfg.name, len(items), params)
    return items, params, desc


def time_oracle(items, params, min_seconds: float, max_passes: int):
    from oracle import aggregator as A
    passes, elapsed, used = 0, 0.0, 1
    while passes < max_passes and (elapsed < min_seconds or passes == 0):
        t = time.perf_counter()
        _, used = A.run_blocks(items, 0)
        elapsed += time.perf_counter() - t
        passes += 1
    return params * passes / elapsed, used, passes, elapsed


# ------------------------------------------------------------------ block-sharded arm

def sharded_main(args, cfg, config, rank, local_rank, world, device):
    """One workload over `world` ranks: every block is owned by one rank; the
    W shards of a block are read in place from the worker ranks' exported
    buffers, or copied into the owner's staging buffer ahead of the aggregate
    (--transport); no collective in the path.  Total work is fixed: strong
    scaling.  One JSON line per transport."""
    import torch.distributed as dist
    import bench_sharded
    from paper_2204_03211_b200 import binding as B

    def exchange(obj):
        got = [None] * world
        dist.all_gather_object(got, obj)
        return got

    red_dev = device if args.dist_backend == "nccl" else None
    transports = ["inplace", "staged"] if args.transport == "both" else [args.transport]
    for transport in transports:
        wl = bench_sharded.ShardedWorkload(cfg, rank, world, local_rank, exchange, dist.barrier, param_device=device,
                                           transport=transport)
        wl.sh.svc.set_option(B.PS_OPT_OVERLAP, int(not args.in_stream))
        wl.fill(0, device)
        n_sched = max(1, min(args.warmup, 8))
        schedules = [configs.rounds_for(cfg, it, args.ticks) for it in range(n_sched)]
        stream = torch.cuda.Stream(device)

        def step(k, s):
            if transport == "staged":
                wl.stage(s)
                exchange(0)                  # host only: every rank's record call has been made
                wl.wait_staged(s)
            n = wl.step(schedules[k % n_sched], s, key=k % n_sched)
            if not args.in_stream:
                wl.sh.svc.join(s)
            return n

        sampler = ClockSampler(local_rank)
        if rank == 0:
            sampler.start()
        for k in range(args.warmup):
            step(k, stream)
        torch.cuda.synchronize(device)
        if rank == 0:
            sampler.mark()
        l0 = wl.sh.svc.launch_info()["launches"]
        ms, rounds, host_ms = timed(lambda k, s: step(args.warmup + k, s), args.steps, stream, True, red_dev)
        clocks = sampler.stop() if rank == 0 else {}
        launches = wl.sh.svc.launch_info()["launches"] - l0
        per_rank = exchange([wl.owned_params, wl.owned_bytes, launches, wl.nvlink_bytes_per_step])
        if rank == 0:
            value = cfg.num_params * args.steps / (ms * 1e-3)                     # every block once per step, all ranks
            worst = max(r[1] for r in per_rank)
            achieved = worst * args.steps / (ms * 1e-3) / 1e9                     # the most loaded rank's HBM traffic
            peak, peak_kind = measured_peak()
            cfg_out = dict(config)
            cfg_out["parallelism"] = "blocks owned by %d ranks (longest-first partition); transport %s" % (
                world, "in place: the owner's kernel reads the workers' buffers" if transport == "inplace" else
                "staged: the workers copy their shards into the owner's memory ahead of the aggregate")
            print(json.dumps({
                "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "strong",
                "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": cfg_out, "transport": transport,
                "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                             "traffic": None, "peak_source": peak_kind + " copy bandwidth",
                             "note": "most loaded rank; with several GPUs the remote shards cross NVLink (read in "
                                     "place by the kernel, or copied ahead of it), which bounds the step before HBM does"},
                "per_rank": [{"params": r[0], "bytes_per_step": r[1], "launches": r[2],
                              "nvlink_bytes_per_step": r[3]} for r in per_rank],
                "cpu_baseline": None, "e2e": None, "gpu_launches": sum(r[2] for r in per_rank),
                "host_ms_per_step": host_ms / args.steps, "clocks": clocks}))
        wl.close()
    dist.destroy_process_group()
    return 0


# ------------------------------------------------------------------ main

def describe(cfg, args) -> dict:
    """The `config` object of the JSON line: both arms print exactly this."""
    return {"workload": "%s: %d packed jobs, %d params, %d blocks, W=%s, %s arrival in <=%d rounds/step" % (
        cfg.name, len(cfg.jobs), cfg.num_params, sum(len(j.blocks) for j in cfg.jobs),
        sorted({j.num_workers for j in cfg.jobs}), cfg.arrival, args.ticks),
        "l2": "inputs (%.1f GB/step) exceed L2; no flush" % (cfg.bytes_per_round() / 1e9)
              if cfg.bytes_per_round() > 4 * 126e6 else
              "inputs (%.1f MB/step) fit the L2: launch-bound, not an HBM figure" % (cfg.bytes_per_round() / 1e6),
        "launch_mode": "in-stream" if args.in_stream else "overlapped, one ps_join per step"}


def cpu_baseline_all(min_seconds: float):
    """Oracle throughput on a bounded sample of each of the five configurations."""
    out = {}
    for name in sorted(configs.CONFIGS):
        c = configs.CONFIGS[name]()
        full_bpp = c.bytes_per_round() / c.num_params
        # bounded: every job keeps a prefix of its blocks, so that the host generates and the oracle
        # reads about 1.5 GB per configuration
        models = len({j.model for j in c.jobs})
        for job in c.jobs:
            keep, used = [], 0
            for b in job.blocks:
                if keep and (used + b.nelem) * job.bytes_per_elem() > 1.5e9 / models:
                    break
                keep.append(b)
                used += b.nelem
            job.blocks = keep
        items, params, desc = oracle_sample(c, None, max_bytes=3e9)
        v, used, passes, el = time_oracle(items, params, min_seconds, 50)
        out[name] = {"value": v, "unit": UNIT, "cores": used, "sample": "%s, %d passes in %.1f s" % (desc, passes, el),
                     "sample_bytes_per_param": sample_bytes_per_param(c, items, params),
                     "workload_bytes_per_param": full_bpp}
        del items
    return out


def sample_bytes_per_param(cfg, items, params) -> float:
    total = 0
    for (hp, step, shards, p, s0, s1) in items:
        total += sum(g.nbytes for g in shards) + 2 * p.nbytes + 2 * s0.nbytes + (2 * s1.nbytes if s1 is not None else 0)
    return total / max(params, 1)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="C4", choices=sorted(configs.CONFIGS))
    ap.add_argument("--ticks", type=int, default=16, help="rounds per iteration window of the arrival schedule")
    ap.add_argument("--min-seconds", type=float, default=2.0,
                    help="the block of --steps steps is repeated until this much device time has been measured")
    ap.add_argument("--max-blocks", type=int, default=400, help="upper bound on those repetitions")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--e2e-mode", default="mapped", choices=["staged", "mapped"],
                    help="staged: only the e2e leg whose shards are copied into device staging; mapped: "
                         "also a second leg (e2e_mapped) whose pinned shards are pushed as they are and read by "
                         "the kernel over PCIe")
    ap.add_argument("--host-pool-gb", type=float, default=24.0,
                    help="upper bound on the pinned host memory of the end-to-end legs (at least the largest job's shards)")
    ap.add_argument("--jobs", default="", help="comma-separated subset of the workload's jobs (profiling a small case)")
    ap.add_argument("--first-blocks", type=int, default=0, help="keep only the first N blocks of every job")
    ap.add_argument("--chunk-elems", type=int, default=0, help="PS_OPT_CHUNK_ELEMS (0 = automatic)")
    ap.add_argument("--kernel", type=int, default=0, help="PS_OPT_KERNEL (0 = automatic, 1 = direct loads, 2 = bulk-copy ring)")
    ap.add_argument("--sparse-transport", action="store_true",
                    help="push embedding-like blocks row-sparse (ps_push_rows); changes the bytes moved, "
                         "so it is a separate experiment, not the default metric; implies --no-e2e")
    ap.add_argument("--in-stream", action="store_true",
                    help="enqueue every launch on the caller's stream (PS_OPT_OVERLAP = 0) instead of letting "
                         "the launches of a step overlap on the service's streams and joining once per step")
    ap.add_argument("--no-split", action="store_true", help="PS_OPT_SPLIT = 0: a large set of ready blocks is one launch")
    ap.add_argument("--no-batch", action="store_true", help="PS_OPT_BATCH = 0: one launch per round, never packed")
    ap.add_argument("--streams", type=int, default=0, help="PS_OPT_WORK_STREAMS (0 = the library's default)")
    ap.add_argument("--unprepared", action="store_true",
                    help="call ps_round with the full argument lists every round instead of ps_round_run on "
                         "rounds prepared once")
    ap.add_argument("--no-pdl", action="store_true", help="PS_OPT_PDL = 0: plain launches for small rounds")
    ap.add_argument("--shard-blocks", action="store_true",
                    help="with --gpus N > 1: ONE workload whose blocks are owned by the N ranks (strong scaling; "
                         "shards are read in place from the worker ranks' exported buffers) instead of N replicas")
    ap.add_argument("--transport", default="both", choices=["inplace", "staged", "both"],
                    help="with --shard-blocks: how a block's shards reach its owner (one JSON line per transport)")
    ap.add_argument("--migration", action="store_true",
                    help="instead of the aggregation benchmark: the overhead of migrating all blocks of a model "
                         "between two contexts (bench_migration.py; its options follow)")
    ap.add_argument("--models", default="alexnet,vgg16,awd_lm,bert_base")
    ap.add_argument("--workers", type=int, default=2)
    ap.add_argument("--reps", type=int, default=7)
    ap.add_argument("--one-by-one", action="store_true", help="--migration: one ps_migrate_block call per block")
    ap.add_argument("--dist-backend", default="nccl", choices=["nccl", "gloo"],
                    help="process-group backend for the barriers and the max over ranks")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-cpu-baseline-all", action="store_true",
                    help="skip timing the oracle on a bounded sample of each of the five configurations")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)
    if args.migration:
        import bench_migration
        if not torch.cuda.is_available():
            raise SystemExit("needs a CUDA device")
        torch.cuda.set_device(0)
        for m in args.models.split(","):
            print(json.dumps(bench_migration.one_model(m, args.workers, args.reps, args.one_by_one)))
        return 0

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    cfg = configs.CONFIGS[args.workload]()
    if args.jobs:
        cfg.jobs = [cfg.jobs[int(x)] for x in args.jobs.split(",")]
        cfg.name += "[jobs %s]" % args.jobs
    if args.first_blocks:
        for job in cfg.jobs:
            job.blocks = job.blocks[:args.first_blocks]
        cfg.name += "[first %d blocks]" % args.first_blocks
    config = describe(cfg, args)

    if args.impl == "reference":
        # The only reference this path has is the CPU oracle: timed as it stands on the host cores,
        # each step one aggregate of a bounded sample of the workload.
        if rank != 0:
            return 0
        items, params, desc = oracle_sample(cfg)
        from oracle import aggregator as A
        for _ in range(args.warmup):
            A.run_blocks(items, 0)
        t = time.perf_counter()
        used = 1
        for _ in range(args.steps):
            _, used = A.run_blocks(items, 0)
        dt = time.perf_counter() - t
        val = params * args.steps / dt
        print(json.dumps({
            "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic", "config": config,
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": used, "kind": "oracle", "sample": desc,
                             "sample_bytes_per_param": sample_bytes_per_param(cfg, items, params),
                             "workload_bytes_per_param": cfg.bytes_per_round() / cfg.num_params},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}))
        return 0

    import torch.distributed as dist
    dist_on = world > 1
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the aggregation path has no CPU fallback")
    local_rank %= torch.cuda.device_count()
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if dist_on:
        if args.dist_backend == "nccl":
            dist.init_process_group("nccl", device_id=device)
        else:
            dist.init_process_group("gloo")
    if args.shard_blocks and dist_on:
        return sharded_main(args, cfg, config, rank, local_rank, world, device)

    # the clocks are sampled from before the warm-up, so that even a short timed region has samples
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()

    n_sched = max(1, min(args.warmup, 8))      # every schedule runs once before the timed region
    wl = Workload(cfg, local_rank, args.ticks, n_sched, sparse=args.sparse_transport, prepared=not args.unprepared)
    B = wl.B
    if args.sparse_transport:
        args.no_e2e = True
        config["transport"] = "row-sparse pushes for embedding tables: %.2f GB of gradient reads avoided per step" % (
            wl.sparse_saved / 1e9)
    wl.svc.set_option(B.PS_OPT_CHUNK_ELEMS, args.chunk_elems)
    wl.svc.set_option(B.PS_OPT_KERNEL, args.kernel)
    wl.svc.set_option(B.PS_OPT_PDL, int(not args.no_pdl))
    wl.svc.set_option(B.PS_OPT_BATCH, int(not args.no_batch))
    wl.svc.set_option(B.PS_OPT_SPLIT, int(not args.no_split))
    if args.streams:
        wl.svc.set_option(B.PS_OPT_WORK_STREAMS, args.streams)
    wl.overlap = not args.in_stream
    wl.svc.set_option(B.PS_OPT_OVERLAP, int(wl.overlap))
    stream = torch.cuda.Stream(device)

    for k in range(args.warmup):
        wl.step(k, stream)
    torch.cuda.synchronize(device)
    if rank == 0:
        sampler.mark()
    stats0 = wl.svc.launch_stats()
    red_dev = device if args.dist_backend == "nccl" else None      # where the max over ranks is reduced
    blocks, rounds, host_ms = timed_blocks(lambda k, s: wl.step(args.warmup + k, s), args.steps, stream, dist_on,
                                           red_dev, args.min_seconds, args.max_blocks)
    clocks = sampler.stop() if rank == 0 else {}
    stats1 = wl.svc.launch_stats()
    info = wl.svc.launch_info()
    ms = statistics.median(blocks)                                   # one block of exactly --steps steps
    value = whole_job_value(wl.params_per_step, world, args.steps, ms)
    achieved = wl.bytes_per_step * args.steps / (ms * 1e-3) / 1e9     # per GPU
    peak, peak_kind = measured_peak()
    # the kernels of the timed region: launches and algorithmic bytes per variant
    mix = []
    for v0, v1 in zip(stats0, stats1):
        n, by = v1["launches"] - v0["launches"], v1["bytes"] - v0["bytes"]
        if n:
            mix.append({"kernel": v1["kernel"], "launches": n, "bytes": by})
    total_bytes = sum(m["bytes"] for m in mix) or 1
    for m in mix:
        m["byte_share"] = m["bytes"] / total_bytes
    dominant = max(mix, key=lambda m: m["bytes"]) if mix else {"kernel": "none", "launches": 0, "bytes": 0}
    launches = sum(m["launches"] for m in mix)
    per_launch_bytes = dominant["bytes"] / max(dominant["launches"], 1)
    # the dominant kernel's average launch duration: the timed region's device time, less nothing —
    # its launches fill the region (other variants' byte share is printed beside it)
    dom_ms = sum(blocks) * dominant.get("byte_share", 1.0) / max(dominant["launches"], 1)
    sha = kernel_sha(dominant["kernel"])
    traffic = None
    captured = NCU_TRAFFIC.get(dominant["kernel"])
    if captured and captured["kernel_sha"] == sha:
        traffic = per_launch_bytes * captured["dram_bytes_per_algorithmic_byte"]

    e2e = e2e_mapped = None
    if not args.no_e2e:
        wl.prepare_host(int(args.host_pool_gb * (1 << 30)))

        def host_leg(host_step, mode):
            host_step(0, stream)        # warm-up (staged: allocates the staging buffers)
            torch.cuda.synchronize(device)
            ems, _, _ = timed(host_step, args.e2e_steps, stream, dist_on, red_dev)
            return {"value": whole_job_value(wl.params_per_step, world, args.e2e_steps, ems), "unit": UNIT,
                    "h2d_bytes_per_step": wl.h2d, "d2h_bytes_per_step": wl.d2h, "steps": args.e2e_steps,
                    "ms_per_step": ems / args.e2e_steps, "mode": mode, "host_pool_bytes": wl.pool_bytes,
                    "h2d_gbs": wl.h2d * args.e2e_steps / (ems * 1e-3) / 1e9}

        # staged: the round's shards are copied from pinned memory into device staging, then the kernel
        # reads the staging; mapped: the pinned shards themselves are pushed (ps_push) and the kernel
        # reads them over PCIe in place.  Same bytes cross the link every step in both.
        e2e = host_leg(wl.step_host, "staged: host shards copied to device staging, then aggregate")
        if args.e2e_mode == "mapped":
            e2e_mapped = host_leg(wl.step_host_mapped, "mapped: ps_push of pinned host pointers, the kernel reads over PCIe")

    cpu = cpu_all = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        items, params, desc = oracle_sample(cfg, wl.slabs)
        v, used, passes, el = time_oracle(items, params, 12.0, 1000)
        cpu = {"value": v, "unit": UNIT, "cores": used, "kind": "oracle",
               "sample": "%s, %d passes in %.1f s" % (desc, passes, el),
               "sample_bytes_per_param": sample_bytes_per_param(cfg, items, params),
               "workload_bytes_per_param": cfg.bytes_per_round() / cfg.num_params}
        del items
        if not args.no_cpu_baseline_all:
            cpu_all = cpu_baseline_all(2.0)

    if rank == 0:
        frac_nominal = achieved / 8000.0
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": config,
            "timed_region": {"blocks": len(blocks), "steps_per_block": args.steps, "ms_per_step": "median block",
                             "ms_per_step_min": min(blocks) / args.steps, "ms_per_step_max": max(blocks) / args.steps,
                             "seconds": sum(blocks) / 1e3, "rounds": rounds, "launches": launches},
            "hbm_gbs_algorithmic": achieved,
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                         "frac": achieved / peak, "traffic": traffic,
                         "peak_source": peak_kind + " copy bandwidth (half reads, half writes; this path mostly "
                                                    "reads, so the ratio can exceed 1)",
                         "frac_of_nominal_8TBs": frac_nominal, "kernel": dominant["kernel"],
                         "kernel_share": dominant.get("byte_share"), "kernels": mix,
                         "bytes_per_launch": per_launch_bytes, "launch_ms": dom_ms, "kernel_sha": sha,
                         "note": "achieved = algorithmic bytes of a block of steps / its event time (launches of a "
                                 "step overlap and pack; table uploads included); launch_ms = the dominant kernel's "
                                 "share of that time / its launches"},
            "cpu_baseline": cpu, "cpu_baseline_all": cpu_all, "e2e": e2e, "e2e_mapped": e2e_mapped,
            "gpu_launches": launches,
            "launch": {"grid": info["grid"], "block": info["block"]},
            "host_ms_per_step": statistics.median(host_ms) / args.steps, "clocks": clocks,
        }
        print(json.dumps(line))
    wl.svc.close()
    if dist_on:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
