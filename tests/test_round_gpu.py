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


@pytest.mark.parametrize("overlap,pdl,flag,batch", [(1, 1, 1, 1), (1, 1, 1, 0), (1, 0, 1, 0), (1, 1, 0, 1), (0, 1, 1, 1),
                                                    (0, 0, 0, 0)],
                         ids=["overlap-pdl-complete-packed", "overlap-pdl-complete", "overlap-plain-complete",
                              "overlap-pdl-ordered", "instream-pdl-complete", "instream-plain-ordered"])
def test_many_small_rounds_in_every_launch_mode(overlap, pdl, flag, batch):
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
        svc.set_option(B.PS_OPT_BATCH, batch)
        flags = B.PS_ROUND_INPUTS_COMPLETE if flag else 0
        stream = torch.cuda.Stream()
        rng = np.random.default_rng(7)
        n_rounds = 0
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
                n_rounds += 1
        svc.join(stream)
        stream.synchronize()
        info = svc.launch_info()
        if overlap and flag and batch:
            assert 4 <= info["launches"] <= n_rounds     # rounds were packed (how many depends on timing)
        else:
            assert info["launches"] == n_rounds
            assert {v["kernel"]: v["launches"] for v in svc.launch_stats()}["ps_aggregate_inline_kernel"] == n_rounds
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
        svc.set_option(B.PS_OPT_SPLIT, 0)         # one launch per round: split, the large round's parts would fit the parameters too
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


@pytest.mark.parametrize("opt,dt", [(configs.SGD, configs.F32), (configs.ADAM, configs.BF16)], ids=["sgd-f32", "adam-bf16"])
def test_prepared_rounds_reuse_their_table_across_iterations_and_survive_migration(opt, dt):
    """The rounds of an iteration are prepared once and run six times from the
    same gradient buffers (refilled in place between iterations).  The cached
    table must follow the step counter (Adam's bias correction changes every
    step) and must be rebuilt when blocks migrate or an option changes."""
    sizes = [70_001, 4096, 33, 300_000, 8193, 1 << 20, 5, 12_345]
    cfg = tiny_config(sizes, 3, opt=opt, grad_dtype=dt)
    cfg.num_contexts = 2
    pair = Pair(cfg)
    svc = pair.svc
    try:
        svc.set_option(B.PS_OPT_OVERLAP, 1)
        stream = torch.cuda.Stream()
        dslab = generate.to_device(generate.grad_slab(cfg, 0, 0), pair.dev)
        groups = [[(0, 0), (0, 1)], [(0, 2)], [(0, 3), (0, 4), (0, 5)], [(0, 6), (0, 7)]]
        rounds = [svc.round_prepare(*_round_args(cfg, dslab, g), g, B.PS_ROUND_INPUTS_COMPLETE) for g in groups]
        out = np.zeros(3, np.uint64)
        for it in range(6):
            slab = generate.grad_slab(cfg, 0, it)
            svc.join(stream)
            stream.synchronize()                          # the previous iteration no longer reads the buffers
            dslab.copy_(generate.to_device(slab, pair.dev))
            torch.cuda.synchronize()
            host = to_np(slab)
            for r, g in zip(rounds, groups):
                svc.round_run(r, stream, out)
                assert [int(x) for x in out[:len(g)]] == [svc.pull(j, b) for (j, b) in g]
                _oracle_round(pair, host, g)
            if it == 1:
                pair.migrate(0, 3, 1 - svc.block_state(0, 3)[2])      # the cached table points at the old place
                pair.migrate(0, 6, 1 - svc.block_state(0, 6)[2])
            if it == 3:
                svc.set_option(B.PS_OPT_CHUNK_ELEMS, 2048)            # another chunking: rebuilt as well
        svc.join(stream)
        stream.synchronize()
        pair.compare()
        for r in rounds:
            svc.round_release(r)
    finally:
        pair.close()


def test_prepared_round_that_is_not_self_contained_takes_outside_pushes():
    """A prepared round may list a task whose pushes (or some of them) arrive
    through ps_push: its table is then built from what was actually pushed."""
    cfg = tiny_config([50_000, 20_000], 2)
    pair = Pair(cfg)
    svc = pair.svc
    try:
        a = generate.to_device(generate.grad_slab(cfg, 0, 0), pair.dev)
        b = generate.to_device(generate.grad_slab(cfg, 0, 1), pair.dev)
        both = [(0, 0), (0, 1)]
        # the round itself pushes block 0 only; block 1's shards come from outside, from another buffer each time
        r = svc.round_prepare(*_round_args(cfg, a, [(0, 0)]), both, B.PS_ROUND_INPUTS_COMPLETE)
        torch.cuda.synchronize()
        for it, other in enumerate((a, b, a)):
            blk = cfg.jobs[0].blocks[1]
            for w in range(2):
                svc.push(0, 1, w, generate.shard_ptr(other, w, blk.job_offset))
            svc.round_run(r, None)
            ha, ho = to_np(a.cpu()), to_np(other.cpu())
            b0 = cfg.jobs[0].blocks[0]
            for w in range(2):
                pair.ora.push(0, 0, w, ha[w, b0.job_offset:b0.job_offset + b0.nelem])
                pair.ora.push(0, 1, w, ho[w, blk.job_offset:blk.job_offset + blk.nelem])
            pair.ora.aggregate(both)
        torch.cuda.synchronize()
        pair.compare()
    finally:
        pair.close()


@pytest.mark.parametrize("prepared", [False, True], ids=["ps_round", "prepared"])
def test_rounds_held_back_behind_a_busy_device_are_packed_and_lose_nothing(prepared):
    """A long launch keeps the device busy; the rounds issued meanwhile are
    held back and leave as a few packed launches.  A block that becomes ready
    again while its previous aggregate still waits in the batch, a statistics
    read and a migration in the middle all force the batch out first."""
    big = 1 << 24
    sizes = [big, big] + [5000 + 17 * k for k in range(30)]
    cfg = tiny_config(sizes, 2)
    cfg.num_contexts = 2
    pair = Pair(cfg)
    svc = pair.svc
    try:
        svc.set_option(B.PS_OPT_OVERLAP, 1)
        stream = torch.cuda.Stream()
        slabs = [generate.grad_slab(cfg, 0, it) for it in range(3)]
        dslabs = [generate.to_device(sl, pair.dev) for sl in slabs]
        hosts = [to_np(sl) for sl in slabs]
        torch.cuda.synchronize()
        flag = B.PS_ROUND_INPUTS_COMPLETE
        before = svc.launch_info()["launches"]
        # prepared rounds read the same buffers every iteration: one slab, refilled between iterations
        rid = [svc.round_prepare(*_round_args(cfg, dslabs[0], [(0, b)]), [(0, b)], flag) for b in range(32)] if prepared else None
        for it in range(3):
            if prepared and it:
                svc.join(stream)
                stream.synchronize()
                dslabs[0].copy_(dslabs[it])
                torch.cuda.synchronize()
            # the device side of the whole iteration first (the oracle is slow: interleaved with
            # it the device would be idle at every round and nothing would ever be held back)
            seen = None
            for b in range(32):                   # blocks 0 and 1 are long launches: the device is busy from here on
                ready = [(0, b)]
                if prepared:
                    svc.round_run(rid[b], stream)
                else:
                    svc.round(*_round_args(cfg, dslabs[it], ready), ready, flag, stream)
                if it == 1 and b == 10:
                    seen = svc.block_stats(0, 5)              # block 5 may still sit in the batch
                if it == 1 and b == 20:
                    svc.migrate_block(0, 15, 1 - svc.block_state(0, 15)[2])
            for b in range(32):
                _oracle_round(pair, hosts[it], [(0, b)])
            if it == 1:
                pair.ora.migrate_block(0, 15, 1 - pair.ora.blocks[(0, 15)].ctx)
                rsq, rstep = pair.ora.block_stats(0, 5)
                assert seen[1] == rstep == 2 and abs(seen[0] - rsq) <= 1e-5 * rsq
        svc.join(stream)
        stream.synchronize()
        launches = svc.launch_info()["launches"] - before
        assert launches < 3 * 32, "nothing was packed: %d launches for %d rounds" % (launches, 3 * 32)
        pair.compare()
        # ps_flush sends a held-back round out without a join
        if prepared:
            dslabs[0].copy_(generate.to_device(slabs[0], pair.dev))
            torch.cuda.synchronize()
        ready = [(0, 0)]
        svc.round(*_round_args(cfg, dslabs[0], ready), ready, flag, stream)
        for b in (2, 3, 4):
            svc.round(*_round_args(cfg, dslabs[0], [(0, b)]), [(0, b)], flag, stream)
        svc.flush()
        torch.cuda.synchronize()
        _oracle_round(pair, hosts[0], [(0, 0), (0, 2), (0, 3), (0, 4)])
        pair.compare()
    finally:
        pair.close()


def test_four_host_threads_each_drive_a_job_through_the_same_service():
    """Many jobs' Agents talk to one Aggregator at once (paper, Section 3.1): four host
    threads, one per job, each with its own stream, send their job's rounds (three
    blocks at a time, inputs complete) for three iterations with no coordination
    between them; calls are serialised inside the service, rounds of different jobs
    interleave and pack as they come.  Every element of every block must come out as
    the oracle's, whatever the interleaving was."""
    import threading
    from helpers import FullPair
    jobs = [tiny_config([70001, 5, 4096, 300000, 33, 1 << 20, 12289], 3).jobs[0],
            tiny_config([1 << 18, 12289, 1, 8192, 555555], 4, opt=configs.ADAM, grad_dtype=configs.BF16).jobs[0],
            tiny_config([2_000_003, 64, 4099], 8, momentum=0.0).jobs[0],
            tiny_config([100000] * 9, 2, opt=configs.ADAM, weight_decay=1e-2).jobs[0]]
    cfg = configs.Config("threads", 77, 3, jobs)
    pair = FullPair(cfg)
    svc = pair.svc
    iters = 3
    try:
        slabs = [[generate.grad_slab(cfg, j, it, pair.dev) for it in range(iters)] for j in range(len(jobs))]
        torch.cuda.synchronize()
        errors, start = [], threading.Barrier(len(jobs))

        def agent(j):
            try:
                job, stream = cfg.jobs[j], torch.cuda.Stream()
                start.wait()
                for it in range(iters):
                    blocks = [b.block for b in job.blocks]
                    for k in range(0, len(blocks), 3):
                        ready = [(j, b) for b in blocks[k:k + 3]]
                        js, bs, ws, ps = [], [], [], []
                        for (_, b) in ready:
                            for w in range(job.num_workers):
                                js.append(j); bs.append(b); ws.append(w)
                                ps.append(generate.shard_ptr(slabs[j][it], w, job.blocks[b].job_offset))
                        svc.round(np.array(js, np.int32), np.array(bs, np.int32), np.array(ws, np.int32),
                                  np.array(ps, np.uint64), ready, B.PS_ROUND_INPUTS_COMPLETE, stream)
                    if it == 1:
                        svc.join(stream)            # one agent joining flushes what the others have queued: allowed
                svc.join(stream)
                stream.synchronize()
            except Exception as e:      # noqa: BLE001
                errors.append((j, e))

        threads = [threading.Thread(target=agent, args=(j,)) for j in range(len(jobs))]
        [t.start() for t in threads]
        [t.join() for t in threads]
        assert not errors, errors
        for it in range(iters):
            for j, job in enumerate(cfg.jobs):
                host = to_np(slabs[j][it])
                ready = []
                for b in job.blocks:
                    for w in range(job.num_workers):
                        pair.ora.push(j, b.block, w, host[w, b.job_offset:b.job_offset + b.nelem])
                    ready.append((j, b.block))
                pair.ora.aggregate(ready)
        assert pair.compare(iters) == cfg.num_params
    finally:
        pair.close()
