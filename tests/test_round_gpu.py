"""ps_round — push, aggregate and pull of one round in a single call — and the
launch machinery behind small rounds: completion words instead of events,
launches that follow an unfinished one on its own stream, programmatic
dependent launch.  Every case is compared with the CPU oracle bit for bit."""
import numpy as np
import pytest
import torch

from helpers import Pair, tiny_config, to_np
from paper_2204_03211_b200 import binding as B
from workload import configs, generate

pytestmark = pytest.mark.gpu


def _round_args(cfg, dslab, ready):
    jobs, blocks, workers, ptrs = [], [], [], []
    for (j, b) in ready:
        job = cfg.jobs[j]
        for w in range(job.num_workers):
            jobs.append(j); blocks.append(b); workers.append(w)
            ptrs.append(generate.shard_ptr(dslab, w, job.blocks[b].job_offset))
    return (np.array(jobs, np.int32), np.array(blocks, np.int32), np.array(workers, np.int32),
            np.array(ptrs, np.uint64))


def _oracle_round(pair, host, ready):
    for (j, b) in ready:
        job = pair.cfg.jobs[j]
        blk = job.blocks[b]
        for w in range(job.num_workers):
            pair.ora.push(j, b, w, host[w, blk.job_offset:blk.job_offset + blk.nelem])
    pair.ora.aggregate(list(ready))


@pytest.mark.parametrize("overlap,pdl,flag", [(1, 1, 1), (1, 0, 1), (1, 1, 0), (0, 1, 1), (0, 0, 0)],
                         ids=["overlap-pdl-complete", "overlap-plain-complete", "overlap-pdl-ordered",
                              "instream-pdl-complete", "instream-plain-ordered"])
def test_many_small_rounds_in_every_launch_mode(overlap, pdl, flag):
    """40 blocks of mixed small sizes, aggregated in rounds of 1-3 blocks, four
    iterations back to back without any host wait: far more launches than
    there are table slots or streams, every block aggregated again while its
    previous launch may still be running."""
    sizes = [1, 5, 1000, 4096, 8191, 8192, 8193, 70_001, 300_000, 33] * 4
    cfg = tiny_config(sizes, 3)
    pair = Pair(cfg)
    svc = pair.svc
    try:
        svc.set_option(B.PS_OPT_OVERLAP, overlap)
        svc.set_option(B.PS_OPT_PDL, pdl)
        flags = B.PS_ROUND_INPUTS_COMPLETE if flag else 0
        stream = torch.cuda.Stream()
        rng = np.random.default_rng(7)
        keep = []
        for it in range(4):
            slab = generate.grad_slab(cfg, 0, it)
            dslab = generate.to_device(slab, pair.dev)
            keep.append(dslab)
            host = to_np(slab)
            torch.cuda.synchronize()              # the gradients are complete in memory before they are pushed
            order = list(rng.permutation(len(sizes)))
            while order:
                k = int(rng.integers(1, 4))
                ready = [(0, int(b)) for b in order[:k]]
                order = order[k:]
                out = np.zeros(len(ready), np.uint64)
                svc.round(*_round_args(cfg, dslab, ready), ready, flags, stream, out)
                assert [int(x) for x in out] == [svc.pull(j, b) for (j, b) in ready]
                _oracle_round(pair, host, ready)
        svc.join(stream)
        stream.synchronize()
        info = svc.launch_info()
        assert info["launches"] >= 4 * len(sizes) // 3
        assert {v["kernel"]: v["launches"] for v in svc.launch_stats()}["ps_aggregate_inline_kernel"] == info["launches"]
        pair.compare()
    finally:
        pair.close()


def test_same_blocks_every_round_follow_each_other_without_events():
    """One job whose whole model is one round: iteration t+1's launch has to
    follow iteration t's.  In overlap mode it goes to the same service stream,
    so the dependency is stream order; results after 12 iterations with no host
    wait in between are the oracle's."""
    cfg = tiny_config([65_536] * 16, 4)
    pair = Pair(cfg)
    svc = pair.svc
    try:
        svc.set_option(B.PS_OPT_OVERLAP, 1)
        every = configs.rounds_all(cfg)[0]
        stream = torch.cuda.Stream()
        keep = []
        for it in range(12):
            slab = generate.grad_slab(cfg, 0, it)
            dslab = generate.to_device(slab, pair.dev)
            keep.append(dslab)
            torch.cuda.synchronize()
            svc.round(*_round_args(cfg, dslab, every), every, B.PS_ROUND_INPUTS_COMPLETE, stream)
            _oracle_round(pair, to_np(slab), every)
        svc.join(stream)
        stream.synchronize()
        pair.compare()
    finally:
        pair.close()


def test_small_and_large_launches_interleave():
    """Rounds that fit the kernel parameters and rounds that upload their table
    (the persistent kernel) alternate on the same blocks in overlap mode."""
    cfg = tiny_config([1 << 22, 3000, 1 << 20, 17, 500_000, 2048] * 4, 2)      # the large round: 2808 chunks
    pair = Pair(cfg)
    svc = pair.svc
    try:
        svc.set_option(B.PS_OPT_OVERLAP, 1)
        every = configs.rounds_all(cfg)[0]
        small = [t for t in every if cfg.jobs[0].blocks[t[1]].nelem <= 3000]
        big = [t for t in every if t not in small]
        stream = torch.cuda.Stream()
        keep = []
        for it in range(5):
            slab = generate.grad_slab(cfg, 0, it)
            dslab = generate.to_device(slab, pair.dev)
            keep.append(dslab)
            host = to_np(slab)
            torch.cuda.synchronize()
            for ready in (small[:3], big, small[3:]) if it % 2 else (big[:2], small, big[2:]):
                svc.round(*_round_args(cfg, dslab, ready), ready, B.PS_ROUND_INPUTS_COMPLETE, stream)
                _oracle_round(pair, host, ready)
        svc.join(stream)
        stream.synchronize()
        kinds = {v["kernel"]: v["launches"] for v in svc.launch_stats()}
        assert kinds["ps_aggregate_inline_kernel"] > 0 and kinds["ps_aggregate_ldg_kernel"] > 0
        pair.compare()
    finally:
        pair.close()


def test_round_without_the_flag_waits_for_the_producer_on_the_callers_stream():
    """The gradients are produced by work enqueued on the caller's stream right
    before the round (a long chain of device copies): without
    PS_ROUND_INPUTS_COMPLETE the launch is ordered after it."""
    n = 1 << 18
    cfg = tiny_config([n], 2)
    pair = Pair(cfg)
    svc = pair.svc
    try:
        svc.set_option(B.PS_OPT_OVERLAP, 1)
        stream = torch.cuda.Stream()
        slab = generate.grad_slab(cfg, 0, 0)
        src = generate.to_device(slab, pair.dev)
        dst = torch.zeros_like(src)
        junk = [torch.empty(64 << 20, dtype=torch.uint8, device=pair.dev) for _ in range(2)]
        torch.cuda.synchronize()
        with torch.cuda.stream(stream):
            for _ in range(20):
                junk[1].copy_(junk[0])            # keeps the stream busy for a few hundred microseconds
            dst.copy_(src)                        # the producer of the gradients
        ready = [(0, 0)]
        svc.round(*_round_args(cfg, dst, ready), ready, 0, stream)
        _oracle_round(pair, to_np(slab), ready)
        svc.join(stream)
        stream.synchronize()
        pair.compare()
    finally:
        pair.close()


def test_stats_and_pull_host_wait_for_a_launch_that_has_no_event():
    cfg = tiny_config([200_000, 64], 4)
    pair = Pair(cfg)
    svc = pair.svc
    try:
        svc.set_option(B.PS_OPT_OVERLAP, 1)
        every = configs.rounds_all(cfg)[0]
        slab = generate.grad_slab(cfg, 0, 0)
        dslab = generate.to_device(slab, pair.dev)
        torch.cuda.synchronize()
        svc.round(*_round_args(cfg, dslab, every), every, B.PS_ROUND_INPUTS_COMPLETE, None)
        _oracle_round(pair, to_np(slab), every)
        # no join, no synchronize: both calls have to find the launch themselves
        sq, step = svc.block_stats(0, 0)
        rsq, rstep = pair.ora.block_stats(0, 0)
        assert step == rstep == 1 and abs(sq - rsq) <= 1e-5 * rsq
        out = torch.empty(64).pin_memory()
        side = torch.cuda.Stream()
        svc.pull_host(0, 1, out, side)
        side.synchronize()
        assert np.array_equal(out.numpy(), pair.ora.pull(0, 1))
        pair.compare()
    finally:
        pair.close()
