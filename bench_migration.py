"""Overhead of migrating ALL blocks of a job to another Aggregator context.

    python bench.py --migration [--models alexnet,vgg16,awd_lm,bert_base] [--workers 2]

The paper's counterpart is its table "Time overhead of migrating all tensors in
a model" (Appendix B): what the training job sees when every tensor of a model
moves while the job runs.  Here the move is a device-to-device copy between two
context arenas of one GPU, enqueued on a side stream right after an iteration's
aggregate; the next iteration's aggregate waits only for the copies of the
blocks it touches.  Reported per model:

  copy_ms     device time of the copies alone (side stream, nothing else running)
  exposed_ms  extra time of "aggregate, migrate everything, aggregate again"
              over "aggregate, aggregate" — the part of the move the job sees
              when the next update follows immediately (no idle window to hide it)
  chain_ms    device time per move when three moves (there, back, there) are
              enqueued back to back: the host part of call k+1 (reserving the
              destination ranges, building the range table) runs while the copy
              of call k is still on the device, as it does when several jobs'
              models move in a row; copy_ms is the cold case, one call on an
              idle stream, host part included
  host_ms     host time inside one ps_migrate_blocks call
  hidden_ms   extra time of the first aggregate AFTER a completed move over an
              ordinary aggregate (the paper's case: the window between the last
              Pull and the next Update hides the copy) — expected about zero

Prints one JSON object per model.  Uses synthetic gradients of the model's shapes.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2204_03211_b200 import binding as B  # noqa: E402
from workload import configs, generate  # noqa: E402


def one_model(model: str, workers: int, reps: int, one_by_one: bool = False):
    job = configs._job(model, model, workers, lr=0.1, momentum=0.9, weight_decay=1e-4)
    cfg = configs.Config("mig-" + model, 7, 1, [job], num_contexts=2)
    dev = torch.device("cuda", 0)
    # room for the model twice per context: in a chain of moves the ranges a block left are
    # released only once its copy has completed
    arena = 2 * sum(2 * (4 * b.nelem + 256) for b in job.blocks) + (64 << 20)
    svc = B.Service(0, 2, arena)
    j = svc.register_job(**job.hparams())
    p0 = generate.init_params(cfg, 0, dev)
    for b in job.blocks:
        svc.register_block(j, b.block, b.nelem, 0, p0[b.job_offset:b.job_offset + b.nelem])
    slab = generate.grad_slab(cfg, 0, 0, dev)
    ready = [(j, b.block) for b in job.blocks]
    tasks = B.make_tasks(ready)
    jobs = np.array([j for b in job.blocks for w in range(workers)], np.int32)
    blocks = np.array([b.block for b in job.blocks for w in range(workers)], np.int32)
    ws = np.array([w for b in job.blocks for w in range(workers)], np.int32)
    ptrs = np.array([generate.shard_ptr(slab, w, b.job_offset) for b in job.blocks for w in range(workers)], np.uint64)
    main, side = torch.cuda.Stream(), torch.cuda.Stream()

    def aggregate():
        svc.push_batch(jobs, blocks, ws, ptrs)
        svc.aggregate(tasks, main)

    def migrate_all(dst):
        if one_by_one:
            for b in job.blocks:
                svc.migrate_block(j, b.block, dst, side)
        else:
            svc.migrate_blocks(tasks, dst, side)

    def timed(fn):
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(main)
        fn()
        e1.record(main)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)

    ctx = [0]

    def flip():
        ctx[0] ^= 1
        return ctx[0]

    for _ in range(2):                      # warm-up (also of both arenas)
        aggregate()
        migrate_all(flip())
    torch.cuda.synchronize()
    base, exposed, hidden, copy, single, chain, host = [], [], [], [], [], [], []
    for _ in range(reps):
        base.append(timed(lambda: (aggregate(), aggregate())))
        exposed.append(timed(lambda: (aggregate(), migrate_all(flip()), aggregate())))

        # the paper's case: the copies land in the idle window before the next update
        aggregate()
        migrate_all(flip())
        torch.cuda.synchronize()
        hidden.append(timed(aggregate))
        single.append(timed(aggregate))
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(side)
        migrate_all(flip())
        e1.record(side)
        torch.cuda.synchronize()
        copy.append(e0.elapsed_time(e1))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(side)
        t0 = time.perf_counter()
        for _ in range(3):                  # (a fourth would wait for the first: the arenas hold the model twice)
            migrate_all(flip())
        host.append((time.perf_counter() - t0) * 1e3 / 3)
        e1.record(side)
        torch.cuda.synchronize()
        chain.append(e0.elapsed_time(e1) / 3)
    med = lambda v: float(sorted(v)[len(v) // 2])
    moved = sum(2 * ((4 * b.nelem + 255) // 256 * 256) for b in job.blocks)
    out = {"model": model, "params": job.num_params, "blocks": len(job.blocks), "workers": workers,
           "calls": "one ps_migrate_block per block" if one_by_one else "one ps_migrate_blocks", "bytes_moved": moved, "copy_ms": med(copy), "copy_gbs": 2 * moved / med(copy) / 1e6,
           "chain_ms": med(chain), "chain_gbs": 2 * moved / med(chain) / 1e6, "host_ms": med(host),
           "two_aggregates_ms": med(base), "exposed_ms": med(exposed) - med(base),
           "one_aggregate_ms": med(single), "hidden_ms": med(hidden) - med(single)}
    svc.close()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--models", default="alexnet,vgg16,awd_lm,bert_base")
    ap.add_argument("--workers", type=int, default=2)
    ap.add_argument("--reps", type=int, default=7)
    ap.add_argument("--one-by-one", action="store_true", help="one ps_migrate_block call per block")
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device")
    torch.cuda.set_device(0)
    for m in args.models.split(","):
        print(json.dumps(one_model(m, args.workers, args.reps, args.one_by_one)))


if __name__ == "__main__":
    main()
