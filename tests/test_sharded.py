"""Block-sharded deployment (one service per rank, every block owned by one
rank, no collective in the aggregation path).

CPU: the ownership map (balanced, deterministic, identical on every rank) and
the per-rank registry, with two gloo ranks over planning-only services.
GPU: two processes sharing one device, each the owner of half the blocks and
the host of half the workers; shards are read in place from the other
process's exported buffer (CUDA IPC) or copied into the owner's staging buffer
ahead of the aggregate; blocks change owner between two aggregates with no host
waiting for its device in between (export, import and the next aggregate are
ordered by interprocess events and the library's own); every owned block is
compared bit for bit with the CPU oracle.  The two ranks' kernels never wait on
one another: ranks meet in host exchanges, streams wait on events."""
import json
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

import bench_sharded  # noqa: E402
from paper_2204_03211_b200 import binding as B, sharded  # noqa: E402
from workload import configs  # noqa: E402


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _costs(cfg):
    return {(j, b.block): job.bytes_per_elem() * b.nelem for j, job in enumerate(cfg.jobs) for b in job.blocks}


@pytest.mark.parametrize("world", [1, 2, 3, 8])
def test_partition_covers_balances_and_repeats(world):
    cfg = configs.c4()
    costs = _costs(cfg)
    owner = sharded.partition(costs, world)
    assert set(owner) == set(costs) and set(owner.values()) <= set(range(world))
    load = [sum(c for k, c in costs.items() if owner[k] == r) for r in range(world)]
    lower = max(sum(costs.values()) / world, max(costs.values()))
    assert max(load) <= 4.0 / 3.0 * lower + 1e-6              # Graham's bound for heaviest-first
    assert max(load) <= 1.01 * lower                          # and much better on 1623 blocks
    shuffled = dict(sorted(costs.items(), key=lambda kv: hash(kv[0]) % 977))
    assert sharded.partition(shuffled, world) == owner        # independent of the order of arrival
    if world == 1:
        assert set(owner.values()) == {0}


def test_partition_small_cases_by_brute_force():
    rng = np.random.default_rng(5)
    for _ in range(30):
        n, world = int(rng.integers(1, 8)), int(rng.integers(1, 4))
        costs = {(0, i): float(rng.integers(1, 50)) for i in range(n)}
        owner = sharded.partition(costs, world)
        got = max(sum(c for k, c in costs.items() if owner[k] == r) for r in range(world))
        best = min(max(sum(c for i, c in enumerate(costs.values()) if (code // world ** i) % world == r)
                       for r in range(world)) for code in range(world ** n))
        assert best <= got <= 4.0 / 3.0 * best + 1e-9


def _cpu_rank(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = configs.c2()
    owner = sharded.partition(_costs(cfg), world)
    sh = sharded.ShardedService(rank, world, B.PS_DEVICE_NONE, 1, 1 << 32)
    sh.set_owners(owner)
    for j, job in enumerate(cfg.jobs):
        assert sh.register_job(**job.hparams()) == j
        for b in job.blocks:
            assert sh.register_block(j, b.block, b.nelem) == (owner[(j, b.block)] == rank)
    every = configs.rounds_all(cfg)[0]
    mine = sh.owned(every)
    host = np.zeros(4, np.float32)
    for (j, b) in every:
        for w in range(cfg.jobs[j].num_workers):
            assert sh.push(j, b, w, host) == ((j, b) in mine)     # pointer bookkeeping only: no device here
    chunks = sh.svc.plan(mine)                                     # the packed table of this rank's launch
    elems = sum(c.elem_count for c in chunks)
    with pytest.raises(B.PsError) as e:
        sh.aggregate(every)                                        # planning-only services never compute
    assert e.value.status == B.PS_ERR_NO_DEVICE
    foreign = next(k for k in every if k not in mine)
    with pytest.raises(B.PsError):
        sh.pull(*foreign)
    maps = [None] * world
    dist.all_gather_object(maps, sorted(owner.items()))
    counts = [None] * world
    dist.all_gather_object(counts, (len(mine), elems))
    with open(out % rank, "w") as f:
        json.dump({"same": all(m == maps[0] for m in maps), "blocks": [c[0] for c in counts],
                   "elems": [c[1] for c in counts]}, f)
    sh.close()
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_owners_and_split_the_registry(tmp_path):
    out = str(tmp_path / "r%d.json")
    mp.spawn(_cpu_rank, args=(2, _free_port(), out), nprocs=2, join=True)
    cfg = configs.c2()
    for r in range(2):
        got = json.load(open(out % r))
        assert got["same"]
        assert sum(got["blocks"]) == len(cfg.jobs[0].blocks) and min(got["blocks"]) > 0
        assert sum(got["elems"]) == cfg.num_params
        assert abs(got["elems"][0] - got["elems"][1]) <= 0.02 * cfg.num_params


def _gpu_rank(rank, world, port, out, transport="inplace", kernel=0):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from helpers import oracle_hp, tiny_config, to_np
    from oracle import aggregator as A
    from workload import generate
    torch.cuda.set_device(0)                                       # both ranks share the one device

    def exchange(obj):
        got = [None] * world
        dist.all_gather_object(got, obj)
        return got

    a = tiny_config([70001, 5, 4096, 300000, 33], 3).jobs[0]
    b = tiny_config([1 << 18, 12289, 1, 8192], 4, opt=configs.ADAM, grad_dtype=configs.BF16).jobs[0]
    cfg = configs.Config("sharded-tiny", 321, 3, [a, b])
    wl = bench_sharded.ShardedWorkload(cfg, rank, world, 0, exchange, dist.barrier, arena_slack=16 << 20,   # room for adopted blocks
                                       transport=transport)
    if kernel:
        wl.sh.svc.set_option(B.PS_OPT_KERNEL, kernel)
    # the oracle of each rank follows EVERY block (they are tiny), so that a block
    # adopted by this rank half-way has its history
    ora = A.OracleAggregator(1, 0)
    for j, job in enumerate(cfg.jobs):
        assert ora.register_job(oracle_hp(job)) == j
        p0 = generate.init_params(cfg, j)
        for blk in job.blocks:
            ora.register_block(j, blk.block, blk.nelem, 0, p0[blk.job_offset:blk.job_offset + blk.nelem].numpy())
    every = configs.rounds_all(cfg)[0]
    rounds = [every[:4], every[4:]]
    remote_reads, adopted, sent = 0, set(), 0
    stream = torch.cuda.Stream()

    def oracle_iteration(it):
        nonlocal remote_reads
        for j, job in enumerate(cfg.jobs):
            host = to_np(generate.grad_slab(cfg, j, it))
            for blk in job.blocks:
                for w in range(job.num_workers):
                    ora.push(j, blk.block, w, host[w, blk.job_offset:blk.job_offset + blk.nelem])
                    if wl.sh.owns(j, blk.block):
                        remote_reads += int(sharded.worker_rank(w, world) != rank)
        ora.aggregate(every)

    def device_iteration():
        if transport == "staged":
            wl.stage(stream)
            exchange(0)                                            # every rank's record call has been made
            wl.wait_staged(stream)
        assert wl.step(rounds, stream, key=0) >= 1

    for it in range(3):
        wl.fill(it, "cpu")
        device_iteration()
        oracle_iteration(it)
        if it == 1 and transport == "inplace":
            # Every rank hands its two lowest blocks of each job to the other rank RIGHT AFTER enqueueing
            # iteration 1's aggregates, and the next aggregates (the same gradient buffers once more, so that
            # nothing has to be refilled and nobody synchronizes) follow at once: the copies wait for the
            # aggregates, the imports for the exports, the new owner's aggregates for the imports — all on
            # the devices' side.
            owner0 = dict(wl.sh.owner)
            moves = []
            for r in range(world):
                for j in range(len(cfg.jobs)):
                    theirs = sorted(blk for (jj, blk), o in owner0.items() if jj == j and o == r)
                    moves += [(j, blk, 1 - r) for blk in theirs[:2]]
            before = set(wl.sh.owned(every))
            sent = wl.migrate(moves, exchange, stream)
            adopted = set(wl.sh.owned(every)) - before
            device_iteration()
            oracle_iteration(it)
            sent += wl.migrate([(j, blk, 1 - r) for (j, blk, r) in moves[:2]], exchange, stream)   # and two of them back
            device_iteration()
            oracle_iteration(it)
        torch.cuda.synchronize()
        dist.barrier()                                             # every rank has read the buffers: refill allowed
    steps_done = 5 if transport == "inplace" else 3
    ok, checked = True, 0
    for (j, blk) in wl.sh.owned(every):
        n = cfg.jobs[j].blocks[blk].nelem
        got = wl.sh.svc.view(wl.sh.pull(j, blk), n).cpu().numpy()
        s0, s1, _ = wl.sh.svc.block_state(j, blk)
        ra, rv = ora.state(j, blk)
        ok &= np.array_equal(got, ora.pull(j, blk))
        ok &= np.array_equal(wl.sh.svc.view(s0, n).cpu().numpy(), ra)
        if rv is not None:
            ok &= np.array_equal(wl.sh.svc.view(s1, n).cpu().numpy(), rv)
        sq, step = wl.sh.svc.block_stats(j, blk)
        rsq, rstep = ora.block_stats(j, blk)
        ok &= step == rstep == steps_done and abs(sq - rsq) <= 1e-5 * abs(rsq) + 1e-300
        checked += 1
    # Pull across ranks: the other rank's blocks, read in place from its mapped arena
    wl.open_arenas(exchange)
    pulled = 0
    for (j, blk) in every:
        if wl.sh.owns(j, blk):
            continue
        n = cfg.jobs[j].blocks[blk].nelem
        raw = sharded.device_bytes(wl.param_address(j, blk), 4 * n, 0).cpu().numpy().view(np.float32)
        ok &= np.array_equal(raw, ora.pull(j, blk))
        pulled += 1
    dist.barrier()
    gone = [k for k in every if not wl.sh.owns(*k)]
    for (j, blk) in gone[:2]:                                      # a block that left is unknown here
        try:
            wl.sh.svc.pull(j, blk)
            ok = False
        except B.PsError as e:
            ok &= e.status == B.PS_ERR_BAD_ARG
    with open(out % rank, "w") as f:
        json.dump({"ok": bool(ok), "checked": checked, "pulled": pulled, "remote_reads": remote_reads, "adopted": len(adopted),
                   "sent": sent, "status": wl.sh.svc.device_status(), "nvlink": wl.nvlink_bytes_per_step}, f)
    wl.close()
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.gpu
def test_two_processes_on_one_device_read_each_others_shards_in_place(tmp_path):
    out = str(tmp_path / "g%d.json")
    mp.spawn(_gpu_rank, args=(2, _free_port(), out), nprocs=2, join=True)
    got = [json.load(open(out % r)) for r in range(2)]
    assert all(g["ok"] and g["status"] == 0 for g in got), got
    assert sum(g["checked"] for g in got) == 9 and min(g["checked"] for g in got) >= 2
    assert all(g["checked"] + g["pulled"] == 9 for g in got)       # the rest was pulled from the other rank's arena
    assert all(g["remote_reads"] > 0 for g in got)                 # each rank consumed shards hosted by the other
    assert all(g["adopted"] >= 2 and g["sent"] > 0 for g in got)   # and blocks changed owner in both directions


@pytest.mark.gpu
def test_two_processes_on_one_device_ring_kernel_reads_mapped_shards(tmp_path):
    """In place again, with the bulk-copy ring kernel: its copies into shared memory
    start at addresses mapped from the other process's buffer (no multicast anywhere)."""
    out = str(tmp_path / "r%d.json")
    mp.spawn(_gpu_rank, args=(2, _free_port(), out, "inplace", 2), nprocs=2, join=True)
    got = [json.load(open(out % r)) for r in range(2)]
    assert all(g["ok"] and g["status"] == 0 for g in got), got
    assert sum(g["checked"] for g in got) == 9 and all(g["remote_reads"] > 0 for g in got)
    assert all(g["adopted"] >= 2 and g["sent"] > 0 for g in got)


@pytest.mark.gpu
def test_two_processes_on_one_device_staged_transport(tmp_path):
    """The same deployment with the workers' shards COPIED into the owner's
    staging buffer ahead of every aggregate (interprocess events order the
    owner's launch after the copies): same results, and the owners' kernels read
    nothing but their own memory."""
    out = str(tmp_path / "s%d.json")
    mp.spawn(_gpu_rank, args=(2, _free_port(), out, "staged"), nprocs=2, join=True)
    got = [json.load(open(out % r)) for r in range(2)]
    assert all(g["ok"] and g["status"] == 0 for g in got), got
    assert sum(g["checked"] for g in got) == 9 and all(g["checked"] + g["pulled"] == 9 for g in got)
    assert all(g["nvlink"] > 0 for g in got)                       # each rank sent shards to the other


@pytest.mark.gpu
def test_bench_block_sharded_arm_two_ranks_on_one_device():
    import subprocess
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", str(_free_port()), os.path.join(ROOT, "bench.py"), "--gpus", "2",
           "--shard-blocks", "--dist-backend", "gloo", "--workload", "C1", "--steps", "5", "--warmup", "3"]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    line = json.loads([l for l in r.stdout.splitlines() if l.startswith("{")][-1])
    cfg = configs.c1()
    assert line["n_gpus"] == 2 and line["scaling"] == "strong" and line["value"] > 0
    assert sum(p["params"] for p in line["per_rank"]) == cfg.num_params
    assert line["gpu_launches"] == sum(p["launches"] for p in line["per_rank"]) == 2 * 5


def test_unregister_and_export_query_on_a_planning_only_service():
    svc = B.Service(device=B.PS_DEVICE_NONE, num_contexts=1, arena_bytes_per_ctx=1 << 20)
    try:
        j = svc.register_job(opt=B.PS_ADAM, grad_dtype=B.PS_F32, num_workers=2, lr=1e-3)
        svc.register_block(j, 3, 1000, 0, None)
        used = svc.arena_info(0)[0]
        assert used == 3 * 4096                                    # p | m | v, each 4000 B rounded up to 256
        assert svc.block_export(j, 3) == (3 * 4096, 0)             # size query: no device needed
        with pytest.raises(B.PsError) as e:
            svc.block_export(j, 3, 1 << 20, 3 * 4096)
        assert e.value.status == B.PS_ERR_NO_DEVICE
        with pytest.raises(B.PsError) as e:
            svc.block_export(j, 3, 1 << 20, 100)                   # destination too small
        assert e.value.status == B.PS_ERR_BAD_ARG
        with pytest.raises(B.PsError) as e:
            svc.block_import(j, 3, 1 << 20, 17, 5)                 # not the block's packed size
        assert e.value.status == B.PS_ERR_BAD_ARG
        svc.unregister_block(j, 3)
        assert svc.arena_info(0)[0] == 0
        for call in (lambda: svc.unregister_block(j, 3), lambda: svc.block_export(j, 3),
                     lambda: svc.push(j, 3, 0, np.zeros(4, np.float32))):
            with pytest.raises(B.PsError) as e:
                call()
            assert e.value.status == B.PS_ERR_BAD_ARG
        svc.register_block(j, 3, 500, 0, None)                     # the id can be used again
        assert svc.block_export(j, 3) == (3 * 2048, 0)
    finally:
        svc.close()


@pytest.mark.gpu
@pytest.mark.parametrize("opt,dt", [(configs.SGD, configs.F32), (configs.ADAM, configs.BF16)])
def test_block_moves_between_two_services_and_training_continues_bit_for_bit(opt, dt):
    """Two services on one device stand for two Aggregators.  A block trains two
    iterations on the first, moves (export -> import -> unregister) and trains
    two more on the second: parameters, state and the step counter (Adam's bias
    correction depends on it) must equal the oracle's four uninterrupted
    iterations."""
    from helpers import Pair, tiny_config, to_np
    from workload import generate
    cfg = tiny_config([70001, 4096], 3, opt=opt, grad_dtype=dt)
    pair = Pair(cfg)
    other = B.Service(0, 1, 8 << 20)
    try:
        job = cfg.jobs[0]
        assert other.register_job(**job.hparams()) == 0
        every = configs.rounds_all(cfg)[0]
        for it in range(2):
            pair.push_iteration(it)
            pair.aggregate(every)
        side = torch.cuda.Stream()
        nbytes, step = pair.svc.block_export(0, 0)
        assert step == 2
        lane = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        assert pair.svc.block_export(0, 0, lane, nbytes, side) == (nbytes, 2)   # ordered after the aggregate
        other.register_block(0, 0, 70001, 0, None)
        other.block_import(0, 0, lane, nbytes, step, side)                   # same stream: after the export
        pair.svc.unregister_block(0, 0)                                       # waits for the export
        with pytest.raises(B.PsError):
            pair.svc.pull(0, 0)
        for it in range(2, 4):
            slab = generate.grad_slab(cfg, 0, it)
            dslab = generate.to_device(slab, "cuda")
            host = to_np(slab)
            for blk in job.blocks:
                svc = other if blk.block == 0 else pair.svc
                for w in range(job.num_workers):
                    svc.push(0, blk.block, w, generate.shard_ptr(dslab, w, blk.job_offset))
                    pair.ora.push(0, blk.block, w, host[w, blk.job_offset:blk.job_offset + blk.nelem])
            # another stream than the import's, and no synchronize in between: the
            # library itself must keep the update behind the copy
            other.aggregate([(0, 0)], torch.cuda.Stream())
            pair.svc.aggregate([(0, 1)])
            pair.ora.aggregate(every)
            torch.cuda.synchronize()
        n = 70001
        s0, s1, _ = other.block_state(0, 0)
        ra, rv = pair.ora.state(0, 0)
        assert np.array_equal(other.view(other.pull(0, 0), n).cpu().numpy(), pair.ora.pull(0, 0))
        assert np.array_equal(other.view(s0, n).cpu().numpy(), ra)
        if rv is not None:
            assert np.array_equal(other.view(s1, n).cpu().numpy(), rv)
        sq, st = other.block_stats(0, 0)
        rsq, rst = pair.ora.block_stats(0, 0)
        assert st == rst == 4 and abs(sq - rsq) <= 1e-5 * rsq
        assert np.array_equal(pair.svc.view(pair.svc.pull(0, 1), 4096).cpu().numpy(), pair.ora.pull(0, 1))
    finally:
        pair.close()
        other.close()


@pytest.mark.gpu
def test_bench_replica_arm_two_ranks_on_one_device():
    """The default arm of bench.py for more than one rank (independent replicas,
    max over ranks, whole-job units), launched the way a multi-GPU run launches
    it; here both ranks share the one device and meet over gloo."""
    import subprocess
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", str(_free_port()), os.path.join(ROOT, "bench.py"), "--gpus", "2",
           "--dist-backend", "gloo", "--workload", "C1", "--steps", "20", "--warmup", "3", "--e2e-steps", "1"]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                                         # rank 0 alone prints
    line = json.loads(lines[0])
    cfg = configs.c1()
    assert line["n_gpus"] == 2 and line["scaling"] == "weak" and line["steps"] == 20
    assert abs(line["value"] - 2 * cfg.num_params / (line["ms_per_step"] * 1e-3)) <= 1e-6 * line["value"]
    assert line["gpu_launches"] == 20 * line["timed_region"]["blocks"] and line["cpu_baseline"] is None
    assert line["e2e"]["h2d_bytes_per_step"] == 4 * 4 * cfg.num_params
