"""Block-sharded deployment (one service per rank, every block owned by one
rank, no collective in the aggregation path).

CPU: the ownership map (balanced, deterministic, identical on every rank) and
the per-rank registry, with two gloo ranks over planning-only services.
GPU: two processes sharing one device, each the owner of half the blocks and
the host of half the workers; shards are read in place from the other
process's exported buffer (CUDA IPC) and every owned block is compared bit for
bit with the CPU oracle.  The two ranks' kernels never wait on one another:
the ranks meet only in host barriers."""
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


def _gpu_rank(rank, world, port, out):
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
    cfg = configs.Config("sharded-tiny", 321, 2, [a, b])
    wl = sharded.ShardedWorkload(cfg, rank, world, 0, exchange, dist.barrier, arena_slack=1 << 20)
    ora = A.OracleAggregator(1, 0)
    for j, job in enumerate(cfg.jobs):
        assert ora.register_job(oracle_hp(job)) == j
        p0 = generate.init_params(cfg, j)
        for blk in job.blocks:
            if wl.sh.owns(j, blk.block):
                ora.register_block(j, blk.block, blk.nelem, 0, p0[blk.job_offset:blk.job_offset + blk.nelem].numpy())
    every = configs.rounds_all(cfg)[0]
    rounds = [every[:4], every[4:]]
    remote_reads = 0
    for it in range(2):
        wl.fill(it, "cpu")
        assert wl.step(rounds, key=0) >= 1
        for j, job in enumerate(cfg.jobs):
            host = to_np(generate.grad_slab(cfg, j, it))
            for blk in job.blocks:
                if not wl.sh.owns(j, blk.block):
                    continue
                for w in range(job.num_workers):
                    ora.push(j, blk.block, w, host[w, blk.job_offset:blk.job_offset + blk.nelem])
                    remote_reads += int(sharded.worker_rank(w, world) != rank)
        ora.aggregate(wl.sh.owned(every))
        torch.cuda.synchronize()
        dist.barrier()                                             # every rank has read the buffers: refill allowed
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
        ok &= step == rstep == 2 and abs(sq - rsq) <= 1e-5 * abs(rsq) + 1e-300
        checked += 1
    with open(out % rank, "w") as f:
        json.dump({"ok": bool(ok), "checked": checked, "remote_reads": remote_reads,
                   "status": wl.sh.svc.device_status()}, f)
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
    assert all(g["remote_reads"] > 0 for g in got)                 # each rank consumed shards hosted by the other


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
