"""Seeded random operation sequences against the service and the oracle side by
side: registrations, dense and row-sparse pushes in any order, aggregates of
random ready subsets on random streams, migrations, blocks that leave the
service (their ids are not reused here: the oracle has no such call), and calls
that must fail without changing anything.  After every aggregate the touched blocks are
compared bit for bit."""
import numpy as np
import pytest
import torch

from oracle import aggregator as A
from paper_2204_03211_b200 import binding as B

pytestmark = pytest.mark.gpu

KINDS = [(B.PS_SGD, B.PS_F32), (B.PS_ADAM, B.PS_F32), (B.PS_SGD, B.PS_BF16), (B.PS_ADAM, B.PS_BF16)]
ROW = 64


def _status(fn, *a):
    try:
        fn(*a)
    except B.PsError as e:
        return e.status
    return 0


@pytest.mark.parametrize("seed", [0, 1, 2, 3])
def test_random_operation_sequences(seed):
    rng = np.random.default_rng(seed)
    nctx = 3
    svc = B.Service(0, nctx, 64 << 20)
    svc.set_option(B.PS_OPT_OVERLAP, seed % 2)          # odd seeds: launches on the service's own streams
    if (seed >> 1) & 1:                                 # seeds 2, 3, 6, 7, ...: the bulk-copy ring kernel
        svc.set_option(B.PS_OPT_KERNEL, 2)
    ora = A.OracleAggregator(nctx)
    streams = [None, torch.cuda.Stream(), torch.cuda.Stream()]
    jobs, blocks = [], {}            # blocks[(j, b)] = dict(n, rows, pushed=set)
    next_id = {}                     # per job: ids handed out so far
    keep = []
    aggregated = 0
    try:
        for step in range(400):
            op = rng.random()
            if not jobs or (op < 0.04 and len(jobs) < 6):
                opt, dt = KINDS[int(rng.integers(4))]
                kw = dict(opt=opt, grad_dtype=dt, num_workers=int(rng.integers(1, 6)),
                          lr=float(rng.choice([0.1, 0.01, 1e-3])), momentum=float(rng.choice([0.0, 0.9])),
                          weight_decay=float(rng.choice([0.0, 1e-2])), grad_scale=float(rng.choice([1.0, 0.5])))
                j = svc.register_job(**kw)
                assert j == ora.register_job(A.HParams(**kw)) == len(jobs)
                jobs.append(kw)
            elif op < 0.12 or not blocks:
                j = int(rng.integers(len(jobs)))
                b = next_id.get(j, 0)
                next_id[j] = b + 1
                rows = int(rng.integers(1, 300))
                n = rows * ROW if rng.random() < 0.6 else int(rng.integers(1, 20000))
                ctx = int(rng.integers(nctx))
                init = rng.normal(0, 0.05, size=n).astype(np.float32)
                svc.register_block(j, b, n, ctx, init)
                ora.register_block(j, b, n, ctx, init)
                blocks[(j, b)] = dict(n=n, pushed=set())
                assert _status(svc.register_block, j, b, n, ctx, init) == B.PS_ERR_DUPLICATE
            elif op < 0.62:
                (j, b), st = list(blocks.items())[int(rng.integers(len(blocks)))]
                W = jobs[j]["num_workers"]
                missing = [w for w in range(W) if w not in st["pushed"]]
                if not missing:
                    assert _status(svc.push, j, b, 0, keep[-1] if keep else 4096) == B.PS_ERR_DUPLICATE
                    continue
                w = int(rng.choice(missing))
                gdt = torch.bfloat16 if jobs[j]["grad_dtype"] == B.PS_BF16 else torch.float32
                n = st["n"]
                g = torch.from_numpy(rng.normal(0, 1e-2, size=n).astype(np.float32)).to(gdt)
                as_np = lambda t: t.view(torch.int16).numpy().view(np.uint16) if gdt == torch.bfloat16 else t.numpy()
                if n % ROW == 0 and rng.random() < 0.5:
                    nrows = n // ROW
                    ids = np.flatnonzero(rng.random(nrows) < 0.3).astype(np.int32)
                    vals = g.view(nrows, ROW)[torch.from_numpy(ids).long()].contiguous()
                    di = torch.from_numpy(ids if len(ids) else np.zeros(1, np.int32)).cuda()
                    dv = (vals if len(ids) else torch.zeros((1, ROW), dtype=gdt)).cuda()
                    keep += [di, dv]
                    svc.push_rows(j, b, w, di, len(ids), ROW, dv)
                    ora.push_rows(j, b, w, ids, ROW, as_np(vals))
                else:
                    d = g.cuda()
                    keep.append(d)
                    svc.push(j, b, w, d)
                    ora.push(j, b, w, as_np(g))
                st["pushed"].add(w)
            elif op < 0.635 and len(blocks) > 3:
                # a block leaves the service (e.g. it moved to another Aggregator): whatever is
                # enqueued for it completes first, its arena range returns, its id is unknown afterwards
                (j, b), st = list(blocks.items())[int(rng.integers(len(blocks)))]
                used = sum(svc.arena_info(c)[0] for c in range(nctx))
                svc.unregister_block(j, b)
                del blocks[(j, b)]
                assert sum(svc.arena_info(c)[0] for c in range(nctx)) < used
                assert _status(svc.pull, j, b) == B.PS_ERR_BAD_ARG
                assert _status(svc.unregister_block, j, b) == B.PS_ERR_BAD_ARG
            elif op < 0.72:
                (j, b), st = list(blocks.items())[int(rng.integers(len(blocks)))]
                dst = int(rng.integers(nctx))
                svc.migrate_block(j, b, dst, streams[int(rng.integers(3))])
                ora.migrate_block(j, b, dst)
            else:
                ready = [k for k, st in blocks.items() if len(st["pushed"]) == jobs[k[0]]["num_workers"]]
                unready = [k for k in blocks if k not in ready]
                if unready and rng.random() < 0.3:
                    bad = ready + [unready[0]]
                    assert _status(svc.aggregate, bad) == B.PS_ERR_NOT_READY      # whole call rejected
                if not ready:
                    continue
                pick = [ready[i] for i in rng.permutation(len(ready))[: int(rng.integers(1, len(ready) + 1))]]
                svc.aggregate(pick, streams[int(rng.integers(3))])
                ora.aggregate(pick)
                aggregated += len(pick)
                for k in pick:
                    blocks[k]["pushed"] = set()
                torch.cuda.synchronize()
                for (j, b) in pick:
                    n = blocks[(j, b)]["n"]
                    s0, s1, ctx = svc.block_state(j, b)
                    assert ctx == ora.blocks[(j, b)].ctx
                    assert np.array_equal(svc.view(svc.pull(j, b), n).cpu().numpy(), ora.pull(j, b)), (step, j, b)
                    assert np.array_equal(svc.view(s0, n).cpu().numpy().view(np.uint32),
                                          ora.state(j, b)[0].view(np.uint32)), (step, j, b)
                    if s1:
                        assert np.array_equal(svc.view(s1, n).cpu().numpy(), ora.state(j, b)[1])
                    sq, t = svc.block_stats(j, b)
                    rsq, rt = ora.block_stats(j, b)
                    assert t == rt and abs(sq - rsq) <= 1e-5 * abs(rsq) + 1e-300
        assert aggregated >= 15 and svc.device_status() == 0
    finally:
        svc.close()


@pytest.mark.parametrize("seed", [10, 11, 12])
def test_random_rounds_with_the_device_kept_busy(seed):
    """The round machinery under a seeded random load, with NO synchronisation
    between operations: one-call rounds with and without the inputs-complete
    flag, prepared rounds, tasks whose pushes arrive partly through ps_push,
    large launches that keep the device busy (so that rounds are held back and
    packed), statistics reads, migrations and explicit flushes in between, and
    calls that must fail without changing anything.  Gradient buffers are never
    rewritten (two fixed sets per block), so nothing but the service's own
    ordering keeps the results right.  Everything is compared with the oracle
    at a few random points and at the end."""
    rng = np.random.default_rng(seed)
    nctx = 2
    svc = B.Service(0, nctx, 1 << 30)
    svc.set_option(B.PS_OPT_OVERLAP, 1)
    ora = A.OracleAggregator(nctx)
    stream = torch.cuda.Stream()
    kinds = [(B.PS_SGD, B.PS_F32, 3), (B.PS_ADAM, B.PS_BF16, 2), (B.PS_SGD, B.PS_F32, 4)]
    sizes = {0: [1, 33, 1000, 4096, 8193, 70_001, 300_000, 12_345, 2048, 65_536, 5, 777],
             1: [64, 5000, 131_072, 9, 40_000, 8192, 1 << 20, 333],
             2: [1 << 24, 1 << 24, 1 << 23]}                     # the large blocks that keep the device busy
    dev, host, nelem, W, count = {}, {}, {}, {}, {}
    try:
        for j, (opt, dt, w) in enumerate(kinds):
            kw = dict(opt=opt, grad_dtype=dt, num_workers=w, lr=1e-2, momentum=0.9 if opt == B.PS_SGD else 0.0,
                      weight_decay=1e-3)
            assert svc.register_job(**kw) == ora.register_job(A.HParams(**kw)) == j
            gdt = torch.bfloat16 if dt == B.PS_BF16 else torch.float32
            for b, n in enumerate(sizes[j]):
                init = rng.normal(0, 0.05, size=n).astype(np.float32)
                ctx = int(rng.integers(nctx))
                svc.register_block(j, b, n, ctx, init)
                ora.register_block(j, b, n, ctx, init)
                nelem[(j, b)], W[(j, b)], count[(j, b)] = n, w, 0
                for s in range(2):
                    for k in range(w):
                        if n >= 1 << 22:                # large: drawn on the device, the oracle gets the same bits
                            tg = torch.Generator(device="cuda").manual_seed(int(rng.integers(1 << 30)))
                            dg = (torch.randn(n, device="cuda", generator=tg) * 1e-2).to(gdt)
                            dev[(j, b, s, k)] = dg
                            g = dg.cpu()
                        else:
                            g = torch.from_numpy(rng.normal(0, 1e-2, size=n).astype(np.float32)).to(gdt)
                            dev[(j, b, s, k)] = g.cuda()
                        host[(j, b, s, k)] = g.view(torch.int16).numpy().view(np.uint16) if gdt == torch.bfloat16 else g.numpy()
        torch.cuda.synchronize()
        small = [k for k in nelem if k[0] != 2]
        big = [k for k in nelem if k[0] == 2]
        partial = {}                                   # block -> workers already pushed through ps_push

        def args_for(keys, skip=None):
            js, bs, ws, ps = [], [], [], []
            for (j, b) in keys:
                s = count[(j, b)] % 2
                for k in range(W[(j, b)]):
                    if skip and k in skip.get((j, b), ()):
                        continue
                    js.append(j); bs.append(b); ws.append(k); ps.append(dev[(j, b, s, k)].data_ptr())
            return (np.array(js, np.int32), np.array(bs, np.int32), np.array(ws, np.int32), np.array(ps, np.uint64))

        todo = []                                      # oracle work, replayed only when something is checked: the
        calls = [0]                                    # host stays fast in between and the device stays busy

        def oracle(keys):
            todo.append(("agg", [(k, count[k] % 2) for k in keys]))
            for k in keys:
                count[k] += 1
            calls[0] += 1

        def catch_up():
            for kind, what in todo:
                if kind == "agg":
                    for (j, b), s in what:
                        for k in range(W[(j, b)]):
                            ora.push(j, b, k, host[(j, b, s, k)])
                    ora.aggregate([k for k, _ in what])
                else:
                    ora.migrate_block(*what)
            todo.clear()

        def compare(keys):
            catch_up()
            svc.join(stream)
            stream.synchronize()
            torch.cuda.synchronize()
            for (j, b) in keys:
                n = nelem[(j, b)]
                s0, s1, ctx = svc.block_state(j, b)
                assert ctx == ora.blocks[(j, b)].ctx
                assert np.array_equal(svc.view(svc.pull(j, b), n).cpu().numpy(), ora.pull(j, b)), (j, b)
                assert np.array_equal(svc.view(s0, n).cpu().numpy(), ora.state(j, b)[0]), (j, b)
                if s1:
                    assert np.array_equal(svc.view(s1, n).cpu().numpy(), ora.state(j, b)[1]), (j, b)
                sq, t = svc.block_stats(j, b)
                rsq, rt = ora.block_stats(j, b)
                assert t == rt == count[(j, b)] and abs(sq - rsq) <= 1e-5 * abs(rsq) + 1e-300

        # prepared rounds over fixed groups; they always read gradient set 0, so they run only at even counts
        groups = [[(0, 0), (0, 1), (0, 2)], [(0, 5), (1, 1)], [(1, 2)], [(0, 9), (0, 10), (1, 5), (1, 7)]]
        prepared = [svc.round_prepare(*args_for(g), g, B.PS_ROUND_INPUTS_COMPLETE) for g in groups]
        rounds = 0
        for step in range(500):
            op = rng.random()
            if op < 0.38:
                free = [k for k in small if k not in partial]
                pick = [free[i] for i in rng.permutation(len(free))[: int(rng.integers(1, 5))]]
                extra = [k for k in partial if rng.random() < 0.5]
                keys = pick + extra
                flags = B.PS_ROUND_INPUTS_COMPLETE if rng.random() < 0.8 else 0
                svc.round(*args_for(keys, partial), keys, flags, stream)
                for k in extra:
                    del partial[k]
                oracle(keys)
                rounds += 1
            elif op < 0.53:
                i = int(rng.integers(len(groups)))
                g = groups[i]
                if any(k in partial for k in g):
                    continue
                if any(count[k] % 2 for k in g):
                    # the round's buffers are set 0; blocks at an odd count take set 1 through a plain round first
                    odd = [k for k in g if count[k] % 2]
                    svc.round(*args_for(odd), odd, B.PS_ROUND_INPUTS_COMPLETE, stream)
                    oracle(odd)
                svc.round_run(prepared[i], stream)
                oracle(g)
                rounds += 1
            elif op < 0.63:
                free = [k for k in small if k not in partial and W[k] > 1]
                k = free[int(rng.integers(len(free)))]
                w = int(rng.integers(W[k]))
                svc.push(k[0], k[1], w, dev[(k[0], k[1], count[k] % 2, w)])
                partial[k] = {w}
            elif op < 0.70:
                k = big[int(rng.integers(len(big)))]
                svc.round(*args_for([k]), [k], B.PS_ROUND_INPUTS_COMPLETE, stream)
                oracle([k])
                rounds += 1
            elif op < 0.76:
                k = small[int(rng.integers(len(small)))]
                sq, t = svc.block_stats(*k)             # a held-back round of this block has to go out first
                catch_up()
                rsq, rt = ora.block_stats(*k)
                assert t == rt == count[k] and abs(sq - rsq) <= 1e-5 * abs(rsq) + 1e-300
            elif op < 0.82:
                k = small[int(rng.integers(len(small)))]
                dst = int(rng.integers(nctx))
                svc.migrate_block(k[0], k[1], dst, stream if rng.random() < 0.5 else None)
                todo.append(("mig", (k[0], k[1], dst)))
            elif op < 0.86:
                svc.flush()
            elif op < 0.93:
                # must fail and change nothing: a worker listed twice; a ready list with an unpushed block
                k = small[int(rng.integers(len(small)))]
                if k in partial:
                    continue
                a = args_for([k])
                dup = tuple(np.concatenate([x, x[:1]]) for x in a)
                assert _status(svc.round, *dup, [k], B.PS_ROUND_INPUTS_COMPLETE, stream) == B.PS_ERR_DUPLICATE
                other = small[(small.index(k) + 1) % len(small)]
                if other not in partial:
                    assert _status(svc.round, *a, [k, other], B.PS_ROUND_INPUTS_COMPLETE, stream) == B.PS_ERR_NOT_READY
            elif op < 0.95:
                compare([small[i] for i in rng.permutation(len(small))[:4]])
        for k in list(partial):                        # finish what is half pushed
            svc.round(*args_for([k], partial), [k], 0, stream)
            oracle([k])
        launches = svc.launch_info()["launches"]
        compare(list(nelem))
        assert rounds >= 150 and svc.device_status() == 0
        assert launches <= calls[0]                    # (how many rounds were held back and packed depends on timing)
    finally:
        svc.close()
