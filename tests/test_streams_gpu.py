"""Ordering across streams, migration failure paths, extreme worker counts."""
import numpy as np
import pytest
import torch

from helpers import Pair, tiny_config, to_np
from paper_2204_03211_b200 import binding as B
from workload import configs, generate

pytestmark = pytest.mark.gpu


def test_same_block_on_alternating_streams_stays_ordered():
    cfg = tiny_config([1 << 20, 70001], 4)
    pair = Pair(cfg)
    try:
        streams = [torch.cuda.Stream(), torch.cuda.Stream(), None]
        every = configs.rounds_all(cfg)[0]
        keep = []
        for it in range(6):
            pair.push_iteration(it)
            keep.append(pair.keep)                      # gradients stay alive: nothing is synchronised in the loop
            pair.svc.aggregate(every, streams[it % 3])
            pair.ora.aggregate(every)
        out = torch.empty(1 << 20).pin_memory()
        s = torch.cuda.Stream()
        pair.svc.pull_host(0, 0, out, s)                # a fourth stream: must wait for the last aggregate
        s.synchronize()
        assert np.array_equal(out.numpy(), pair.ora.pull(0, 0))
        pair.compare()
    finally:
        pair.close()


def test_migration_without_room_fails_cleanly_and_block_keeps_working():
    # blocks 0 and 2 start in context 0, block 1 in context 1 (round-robin); SGD: 2 ranges per block
    cfg = tiny_config([200_000, 100_000, 50_000], 2)
    cfg.num_contexts = 2
    pair = Pair(cfg, arena_bytes=2_500_000)
    svc = pair.svc
    try:
        every = configs.rounds_all(cfg)[0]
        pair.push_iteration(0)
        pair.aggregate(every)
        start = [svc.arena_info(c)[0] for c in range(2)]
        assert start == [1_600_000 + 400_384, 800_256]
        with pytest.raises(B.PsError) as e:
            svc.migrate_block(0, 1, 0)                  # 2,000,384 + 800,256 exceeds the arena
        assert e.value.status == B.PS_ERR_NOMEM
        assert svc.block_state(0, 1)[2] == 1 and [svc.arena_info(c)[0] for c in range(2)] == start
        with pytest.raises(B.PsError) as e:
            svc.migrate_block(0, 0, 5)
        assert e.value.status == B.PS_ERR_BAD_ARG
        svc.migrate_block(0, 0, 0)                      # same context: no-op
        pair.migrate(0, 2, 1)                           # the small block fits beside block 1
        pair.migrate(0, 2, 0)                           # and back, before the first copy was waited for
        pair.push_iteration(1)
        pair.aggregate(every)
        pair.compare()
        torch.cuda.synchronize()
        assert [svc.arena_info(c)[0] for c in range(2)] == start
    finally:
        pair.close()


@pytest.mark.parametrize("dt", [configs.F32, configs.BF16])
@pytest.mark.parametrize("kernel", [1, 2, 3], ids=["ldg", "bulk", "inline"])
def test_maximum_worker_count(dt, kernel):
    # (the ring kernel takes W = 256 in 86 fp32 or 43 bf16 stages per tile)
    cfg = tiny_config([4096 + 3, 9000], B.PS_MAX_WORKERS, grad_dtype=dt, grad_std=1e-3)
    pair = Pair(cfg, kernel=kernel)
    try:
        for it in range(2):
            pair.push_iteration(it)
            pair.aggregate(configs.rounds_all(cfg)[0])
        pair.compare()
    finally:
        pair.close()


def test_destroy_with_work_in_flight():
    cfg = tiny_config([1 << 21], 8)
    pair = Pair(cfg)
    pair.push_iteration(0)
    pair.svc.aggregate([(0, 0)], torch.cuda.Stream())
    pair.close()                                        # waits for the launch, then frees everything
    torch.cuda.synchronize()                            # the context is still healthy
    x = torch.ones(16, device="cuda")
    assert float(x.sum()) == 16.0
    assert B.load().ps_destroy(None) == B.PS_ERR_BAD_HANDLE


def test_one_very_large_block():
    # 2^28 + 5 elements in ONE block: 32,769 chunks, offsets beyond 2^30 bytes, a ragged tail
    n = (1 << 28) + 5
    cfg = tiny_config([n], 1, lr=0.05, momentum=0.5, weight_decay=1e-3)
    pair = Pair(cfg)
    try:
        pair.push_iteration(0)
        pair.aggregate([(0, 0)])
        pair.compare()
    finally:
        pair.close()


def test_concurrent_host_threads_are_serialised_by_the_service():
    import threading
    cfg = tiny_config([50_000] * 8, 4)
    pair = Pair(cfg)
    try:
        slab = generate.grad_slab(cfg, 0, 0)
        dslab = generate.to_device(slab, pair.dev)
        host = to_np(slab)
        job = cfg.jobs[0]
        errors = []

        def worker(w):
            try:
                for b in job.blocks:
                    pair.svc.push(0, b.block, w, generate.shard_ptr(dslab, w, b.job_offset))
            except Exception as e:      # noqa: BLE001
                errors.append(e)

        ts = [threading.Thread(target=worker, args=(w,)) for w in range(4)]
        [t.start() for t in ts]
        [t.join() for t in ts]
        assert not errors
        for b in job.blocks:
            for w in range(4):
                pair.ora.push(0, b.block, w, host[w, b.job_offset:b.job_offset + b.nelem])
        pair.aggregate(configs.rounds_all(cfg)[0])
        pair.compare()
    finally:
        pair.close()


def test_batched_migration_is_all_or_nothing_and_chains_without_host_waits():
    sizes = [300_000, 5, 70_000, 1 << 20, 4096, 123_457] * 20          # 120 blocks: two gather launches per batch
    cfg = tiny_config(sizes, 2)
    cfg.num_contexts = 3
    pair = Pair(cfg)
    svc = pair.svc
    try:
        every = configs.rounds_all(cfg)[0]
        pair.push_iteration(0)
        pair.aggregate(every)
        with pytest.raises(B.PsError) as e:
            svc.migrate_blocks(every + [every[0]], 1)
        assert e.value.status == B.PS_ERR_DUPLICATE
        with pytest.raises(B.PsError) as e:
            svc.migrate_blocks(every, 7)
        assert e.value.status == B.PS_ERR_BAD_ARG
        side = torch.cuda.Stream()
        # everything to context 2, then straight on to context 0 and back to 1: each batch is ordered
        # after the previous one on the device, the host never waits
        for dst in (2, 0, 1):
            svc.migrate_blocks(every, dst, side)
            for (j, b) in every:
                pair.ora.migrate_block(j, b, dst)
        pair.push_iteration(1)
        pair.aggregate(every)                           # default stream: must wait for the last batch
        pair.compare()
        assert all(svc.block_state(0, b)[2] == 1 for _, b in every)
        torch.cuda.synchronize()
        used = [svc.arena_info(c)[0] for c in range(3)]
        assert used[0] == 0 and used[2] == 0 and used[1] > 0          # the sources were released
        # a destination without room for the whole batch: nothing moves
        tiny = B.Service(0, 2, (1 << 20) + (1 << 19))
        try:
            j = tiny.register_job(num_workers=1)
            for b in range(3):
                tiny.register_block(j, b, 60_000, 0)                  # 3 x 480,256 bytes in context 0
            tiny.register_block(j, 3, 60_000, 1)                      # context 1 has room for two more only
            with pytest.raises(B.PsError) as e:
                tiny.migrate_blocks([(j, 0), (j, 1), (j, 2)], 1)
            assert e.value.status == B.PS_ERR_NOMEM
            assert [tiny.block_state(j, b)[2] for b in range(4)] == [0, 0, 0, 1]
            assert tiny.arena_info(1)[0] == 480_256
            tiny.migrate_blocks([(j, 0), (j, 2)], 1)
            assert [tiny.block_state(j, b)[2] for b in range(4)] == [1, 0, 1, 1]
        finally:
            tiny.close()
    finally:
        pair.close()


def test_ring_kernel_gives_up_when_its_wait_limit_runs_out_and_says_so():
    """Every wait inside the bulk-copy kernel is bounded.  With the limit set to
    about a thousand cycles — less than one round trip to HBM — the first
    consumer wait of an otherwise ordinary launch runs out: the kernel records
    it in the status word, lets its copies in flight land and returns promptly;
    the context stays usable and a launch with the default limit on freshly
    registered blocks matches the oracle bit for bit."""
    import time
    cfg = tiny_config([1 << 22] * 4, 8)
    pair = Pair(cfg, kernel=2)
    try:
        pair.svc.set_option(B.PS_OPT_WAIT_CYCLES, 64)
        assert pair.svc.get_option(B.PS_OPT_WAIT_CYCLES) == 64
        pair.push_iteration(0)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        pair.svc.aggregate(configs.rounds_all(cfg)[0])
        status = pair.svc.device_status()                # waits for the device
        assert time.perf_counter() - t0 < 5.0            # no wait inside the kernel outlived its limit by much
        assert status != 0
        assert pair.svc.launch_info()["kernel"] == "bulk"
        with pytest.raises(B.PsError):
            pair.svc.set_option(B.PS_OPT_WAIT_CYCLES, 0)
    finally:
        pair.close()
    x = torch.ones(1 << 20, device="cuda")               # the context is healthy
    assert float(x.sum()) == float(1 << 20)
    again = Pair(cfg, kernel=2)                          # default limit, fresh blocks
    try:
        for it in range(2):
            again.push_iteration(it)
            again.aggregate(configs.rounds_all(cfg)[0])
        assert again.svc.device_status() == 0
        assert again.svc.launch_info()["kernel"] == "bulk"
        again.compare()
    finally:
        again.close()
