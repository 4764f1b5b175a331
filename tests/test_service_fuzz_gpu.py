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
