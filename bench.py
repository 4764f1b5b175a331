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

# DRAM traffic of the dominant kernel from the committed ncu capture
# (profiles/), as measured dram bytes per algorithmic byte, keyed by the hash
# of the kernel source it was taken from.  A changed kernel reports null.
NCU_TRAFFIC = {"kernel_sha": "52e594e26b34", "dram_bytes_per_algorithmic_byte": 0.981}


def kernel_sha() -> str:
    h = hashlib.sha256()
    for name in ("ps_types.cuh", "ps_math.cuh", "ps_rows.cuh", "ps_kernel_ldg.cuh"):
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
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.path = index, None, None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if not self.proc:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 7:
                    continue
                try:
                    sm.append(float(f[0]))
                    mx.append(float(f[1]))
                except ValueError:
                    continue
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            # under load = the upper half of the samples (the sampler also sees set-up and idle gaps)
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


# ------------------------------------------------------------------ our arm

class Workload:
    """The service, the device-resident gradients and the per-round call
    arguments of one workload, prepared outside any timed region."""

    def __init__(self, cfg: configs.Config, device: int, ticks: int, n_schedules: int, sparse: bool = False):
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
        self.params_per_step = cfg.num_params
        self.bytes_per_step = cfg.bytes_per_round() - self.sparse_saved

    def step(self, k: int, stream) -> int:
        """Push, aggregate, pull — device-resident gradients.  Returns launches."""
        # The C entry points are called with arguments marshalled once, outside
        # the timed region (array addresses as integers): one C-ABI call per round
        # (ps_round = push, aggregate, pull), plus one for row-sparse pushes if any.
        lib, h, sp = self.lib, self.svc.handle, int(stream.cuda_stream)
        rounds = self.schedules[k % len(self.schedules)]
        flags = self.round_flags
        for r in rounds:
            rc = 0
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
        total = sum(s.numel() * s.element_size() for s in self.slabs)
        pool_bytes = min(pool_bytes, total)
        self.pool = torch.empty(pool_bytes // 4, dtype=torch.float32).pin_memory()
        # fill the pool with the same gradient bits (device -> host copy of the slabs' head)
        flat = self.pool.view(torch.uint8)
        off = 0
        for s in self.slabs:
            src = (s._base if s._base is not None else s).view(-1).view(torch.uint8)
            n = min(src.numel(), flat.numel() - off)
            if n <= 0:
                break
            flat[off:off + n].copy_(src[:n])
            off += n
        self.out = torch.empty(self.cfg.num_params, dtype=torch.float32).pin_memory()
        self.pool_bytes = pool_bytes
        self.pull_stream = torch.cuda.Stream(torch.device("cuda", self.device))
        self.pull_done = torch.cuda.Event()
        self.h2d = total
        self.d2h = self.cfg.num_params * 4
        self._out_off, acc = {}, 0
        for j, job in enumerate(self.cfg.jobs):
            self._out_off[j] = acc
            acc += job.num_params

    def step_host(self, k: int, stream) -> int:
        svc, cfg = self.svc, self.cfg
        rounds = self.schedules[k % len(self.schedules)]
        pool_ptr, pool_bytes = self.pool.data_ptr(), self.pool_bytes
        cursor = 0
        out_ptr = self.out.data_ptr()
        out_off = {}
        acc = 0
        for j, job in enumerate(cfg.jobs):
            out_off[j] = acc
            acc += job.num_params
        for r in rounds:
            for (j, b) in r["ready"]:
                job = cfg.jobs[j]
                nbytes = job.blocks[b].nelem * (2 if job.grad_dtype == configs.BF16 else 4)
                for w in range(job.num_workers):
                    if cursor + nbytes > pool_bytes:
                        cursor = 0
                    svc.push_host(j, b, w, pool_ptr + cursor, stream)
                    cursor += (nbytes + 255) // 256 * 256
            svc.aggregate(r["tasks"], stream)
            # parameters travel back on a second stream (the library orders each copy after the
            # block's aggregate), so device-to-host traffic overlaps the next round's uploads
            for (j, b) in r["ready"]:
                svc.pull_host(j, b, out_ptr + 4 * (out_off[j] + cfg.jobs[j].blocks[b].job_offset), self.pull_stream)
        self.pull_done.record(self.pull_stream)
        stream.wait_event(self.pull_done)           # the step ends when its last result is on the host
        if self.overlap:
            svc.join(stream)
        return len(rounds)


    def step_host_mapped(self, k: int, stream) -> int:
        """End to end without staging copies: pinned host memory is addressable
        from the device, so the pinned shards are pushed as they are and the
        aggregation kernel reads them over PCIe in place; parameters return to
        the host as in step_host."""
        svc, cfg = self.svc, self.cfg
        rounds = self.schedules[k % len(self.schedules)]
        if not hasattr(self, "_mapped_args"):
            self._mapped_args = {}
        out_ptr = self.out.data_ptr()
        for i, r in enumerate(rounds):
            key = (k % len(self.schedules), i)
            if key not in self._mapped_args:
                # where each (block, worker) shard of this round sits in the pinned pool
                jobs, blocks, workers, ptrs = [], [], [], []
                cursor = 0
                for (j, b) in r["ready"]:
                    job = cfg.jobs[j]
                    nbytes = job.blocks[b].nelem * (2 if job.grad_dtype == configs.BF16 else 4)
                    for w in range(job.num_workers):
                        if cursor + nbytes > self.pool_bytes:
                            cursor = 0
                        jobs.append(j); blocks.append(b); workers.append(w)
                        ptrs.append(self.pool.data_ptr() + cursor)
                        cursor += (nbytes + 255) // 256 * 256
                self._mapped_args[key] = (np.array(jobs, np.int32), np.array(blocks, np.int32),
                                          np.array(workers, np.int32), np.array(ptrs, np.uint64))
            svc.push_batch(*self._mapped_args[key])
            svc.aggregate(r["tasks"], stream)
            for (j, b) in r["ready"]:
                svc.pull_host(j, b, out_ptr + 4 * (self._out_off[j] + cfg.jobs[j].blocks[b].job_offset),
                              self.pull_stream)
        self.pull_done.record(self.pull_stream)
        stream.wait_event(self.pull_done)
        if self.overlap:
            svc.join(stream)
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
    bracketed by barrier + synchronize; returns (ms max over ranks, launches)."""
    import torch.distributed as dist
    torch.cuda.synchronize(device)
    if dist_on:
        dist.barrier()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches = 0
    host0 = time.perf_counter()
    with torch.cuda.stream(stream):
        t0.record(stream)
        for k in range(steps):
            launches += fn(k, stream)
        t1.record(stream)
    host_ms = (time.perf_counter() - host0) * 1e3
    torch.cuda.synchronize(device)
    if dist_on:
        dist.barrier()
    ms = max_over_ranks(t0.elapsed_time(t1), device)
    return ms, launches, host_ms


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
    """One workload over `world` ranks: every block is owned by one rank, the
    W shards of a block are read in place from the worker ranks' exported
    buffers (no collective in the path).  Total work is fixed: strong scaling."""
    import torch.distributed as dist
    from paper_2204_03211_b200 import sharded

    def exchange(obj):
        got = [None] * world
        dist.all_gather_object(got, obj)
        return got

    red_dev = device if args.dist_backend == "nccl" else None
    wl = sharded.ShardedWorkload(cfg, rank, world, local_rank, exchange, dist.barrier, param_device=device)
    from paper_2204_03211_b200 import binding as B
    wl.sh.svc.set_option(B.PS_OPT_OVERLAP, int(not args.in_stream))
    wl.fill(0, device)
    n_sched = max(1, min(args.warmup + args.steps, 8))
    schedules = [configs.rounds_for(cfg, it, args.ticks) for it in range(n_sched)]
    stream = torch.cuda.Stream(device)

    def step(k, s):
        n = wl.step(schedules[k % n_sched], s, key=k % n_sched)
        if not args.in_stream:
            wl.sh.svc.join(s)
        return n

    for k in range(args.warmup):
        step(k, stream)
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    ms, launches, host_ms = timed(lambda k, s: step(args.warmup + k, s), args.steps, stream, True, red_dev)
    clocks = sampler.stop() if rank == 0 else {}
    mine = [wl.owned_params, wl.owned_bytes, launches]
    per_rank = exchange(mine)
    if rank == 0:
        value = cfg.num_params * args.steps / (ms * 1e-3)                     # every block once per step, all ranks
        worst = max(r[1] for r in per_rank)
        achieved = worst * args.steps / (ms * 1e-3) / 1e9                     # the most loaded rank's HBM traffic
        peak, peak_kind = measured_peak()
        config["parallelism"] = "blocks owned by %d ranks (longest-first partition), shards read in place from peers" % world
        config["launch_mode"] = "in-stream" if args.in_stream else "overlapped, one ps_join per step"
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "strong",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": config,
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": None, "peak_source": peak_kind + " copy bandwidth",
                         "note": "most loaded rank; with several GPUs the remote shards arrive over NVLink, "
                                 "which bounds the step before HBM does"},
            "per_rank": [{"params": r[0], "bytes_per_step": r[1], "launches": r[2]} for r in per_rank],
            "cpu_baseline": None, "e2e": None, "gpu_launches": sum(r[2] for r in per_rank),
            "host_ms_per_step": host_ms / args.steps, "clocks": clocks}))
    wl.close()
    dist.destroy_process_group()
    return 0


# ------------------------------------------------------------------ main

def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="C4", choices=sorted(configs.CONFIGS))
    ap.add_argument("--ticks", type=int, default=16, help="rounds per iteration window of the arrival schedule")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--e2e-mode", default="mapped", choices=["staged", "mapped"],
                    help="staged: only the e2e leg whose shards ps_push_host copies into device staging; mapped: "
                         "also a second leg (e2e_mapped) whose pinned shards are pushed as they are and read by "
                         "the kernel over PCIe")
    ap.add_argument("--host-pool-gb", type=float, default=8.0)
    ap.add_argument("--jobs", default="", help="comma-separated subset of the workload's jobs (profiling a small case)")
    ap.add_argument("--max-blocks", type=int, default=0, help="keep only the first N blocks of every job")
    ap.add_argument("--chunk-elems", type=int, default=0, help="PS_OPT_CHUNK_ELEMS (0 = automatic)")
    ap.add_argument("--kernel", type=int, default=0, help="PS_OPT_KERNEL (0 = automatic, 1 = direct loads, 2 = bulk-copy ring)")
    ap.add_argument("--sparse-transport", action="store_true",
                    help="push embedding-like blocks row-sparse (ps_push_rows); changes the bytes moved, "
                         "so it is a separate experiment, not the default metric; implies --no-e2e")
    ap.add_argument("--in-stream", action="store_true",
                    help="enqueue every launch on the caller's stream (PS_OPT_OVERLAP = 0) instead of letting "
                         "the launches of a step overlap on the service's streams and joining once per step")
    ap.add_argument("--shard-blocks", action="store_true",
                    help="with --gpus N > 1: ONE workload whose blocks are owned by the N ranks (strong scaling; "
                         "shards are read in place from the worker ranks' exported buffers) instead of N replicas")
    ap.add_argument("--dist-backend", default="nccl", choices=["nccl", "gloo"],
                    help="process-group backend for the barriers and the max over ranks")
    ap.add_argument("--no-pdl", action="store_true", help="PS_OPT_PDL = 0: plain launches for small rounds")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    cfg = configs.CONFIGS[args.workload]()
    if args.jobs:
        cfg.jobs = [cfg.jobs[int(x)] for x in args.jobs.split(",")]
        cfg.name += "[jobs %s]" % args.jobs
    if args.max_blocks:
        for job in cfg.jobs:
            job.blocks = job.blocks[:args.max_blocks]
        cfg.name += "[first %d blocks]" % args.max_blocks
    config = {"workload": "%s: %d packed jobs, %d params, %d blocks, W=%s, %s arrival in <=%d rounds/step" % (
        cfg.name, len(cfg.jobs), cfg.num_params, sum(len(j.blocks) for j in cfg.jobs),
        sorted({j.num_workers for j in cfg.jobs}), cfg.arrival, args.ticks),
        "l2": "inputs (%.1f GB/step) exceed L2; no flush" % (cfg.bytes_per_round() / 1e9)}

    if args.impl == "reference":
        if rank != 0:
            return 0
        items, params, desc = oracle_sample(cfg)
        from oracle import aggregator as A
        for _ in range(min(args.warmup, 1)):
            A.run_blocks(items, 0)
        t = time.perf_counter()
        used = 1
        for _ in range(args.steps):
            _, used = A.run_blocks(items, 0)
        dt = time.perf_counter() - t
        val = params * args.steps / dt
        print(json.dumps({
            "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": min(args.warmup, 1), "ms_per_step": dt / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic", "config": config,
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": used, "kind": "oracle", "sample": desc},
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

    n_sched = max(1, min(args.warmup + args.steps, 8))
    wl = Workload(cfg, local_rank, args.ticks, n_sched, sparse=args.sparse_transport)
    if args.sparse_transport:
        args.no_e2e = True
        config["transport"] = "row-sparse pushes for embedding tables: %.2f GB of gradient reads avoided per step" % (
            wl.sparse_saved / 1e9)
    wl.svc.set_option(wl.B.PS_OPT_CHUNK_ELEMS, args.chunk_elems)
    wl.svc.set_option(wl.B.PS_OPT_KERNEL, args.kernel)
    wl.svc.set_option(wl.B.PS_OPT_PDL, int(not args.no_pdl))
    wl.overlap = not args.in_stream
    wl.svc.set_option(wl.B.PS_OPT_OVERLAP, int(wl.overlap))
    config["launch_mode"] = "overlapped, one ps_join per step" if wl.overlap else "in-stream"
    stream = torch.cuda.Stream(device)

    for k in range(args.warmup):
        wl.step(k, stream)
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    l0 = wl.svc.launch_info()["launches"]
    red_dev = device if args.dist_backend == "nccl" else None      # where the max over ranks is reduced
    ms, launches, host_ms = timed(lambda k, s: wl.step(args.warmup + k, s), args.steps, stream, dist_on, red_dev)
    clocks = sampler.stop() if rank == 0 else {}
    info = wl.svc.launch_info()
    assert info["launches"] - l0 == launches
    value = whole_job_value(wl.params_per_step, world, args.steps, ms)
    achieved = wl.bytes_per_step * args.steps / (ms * 1e-3) / 1e9     # per GPU
    peak, peak_kind = measured_peak()
    per_launch_bytes = wl.bytes_per_step * args.steps / launches
    sha = kernel_sha()
    traffic = None
    if NCU_TRAFFIC["kernel_sha"] == sha and NCU_TRAFFIC["dram_bytes_per_algorithmic_byte"]:
        traffic = per_launch_bytes * NCU_TRAFFIC["dram_bytes_per_algorithmic_byte"]

    e2e = e2e_mapped = None
    if not args.no_e2e:
        wl.prepare_host(int(args.host_pool_gb * (1 << 30)))
        def host_leg(host_step, mode):
            host_step(0, stream)        # warm-up (staged: allocates the staging buffers)
            torch.cuda.synchronize(device)
            ems, _, _ = timed(host_step, args.e2e_steps, stream, dist_on, red_dev)
            return {"value": whole_job_value(wl.params_per_step, world, args.e2e_steps, ems), "unit": UNIT,
                    "h2d_bytes_per_step": wl.h2d, "d2h_bytes_per_step": wl.d2h, "steps": args.e2e_steps,
                    "ms_per_step": ems / args.e2e_steps, "mode": mode, "host_pool_bytes": wl.pool_bytes}

        # staged: ps_push_host copies every shard from pinned memory into device staging, then the kernel
        # reads the staging; mapped: the pinned shards themselves are pushed (ps_push) and the kernel
        # reads them over PCIe in place.  Same bytes cross the link every step in both.
        e2e = host_leg(wl.step_host, "staged: ps_push_host copies, then aggregate")
        if args.e2e_mode == "mapped":
            e2e_mapped = host_leg(wl.step_host_mapped, "mapped: ps_push of pinned host pointers, the kernel reads over PCIe")

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        items, params, desc = oracle_sample(cfg, wl.slabs)
        v, used, passes, el = time_oracle(items, params, 12.0, 1000)
        cpu = {"value": v, "unit": UNIT, "cores": used, "kind": "oracle",
               "sample": "%s, %d passes in %.1f s" % (desc, passes, el)}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": config,
            "hbm_gbs_algorithmic": achieved,
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                         "frac": achieved / peak, "traffic": traffic, "peak_source": peak_kind + " copy bandwidth",
                         "frac_of_nominal_8TBs": achieved / 8000.0, "kernel": info["kernel"],
                         "bytes_per_launch": per_launch_bytes, "kernel_sha": sha,
                         "note": "duration = event time of the whole timed region / launches "
                                 "(launches of a step may overlap; table uploads included)"},
            "cpu_baseline": cpu, "e2e": e2e, "e2e_mapped": e2e_mapped, "gpu_launches": launches,
            "launch": {"grid": info["grid"], "block": info["block"]},
            "host_ms_per_step": host_ms / args.steps, "clocks": clocks,
        }
        print(json.dumps(line))
    wl.svc.close()
    if dist_on:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
