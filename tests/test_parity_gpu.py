"""CUDA path vs CPU oracle, element by element, through the C ABI."""
import numpy as np
import pytest
import torch

from helpers import Pair, tiny_config, to_np, assert_close
from paper_2204_03211_b200 import binding as B
from workload import configs, generate

pytestmark = pytest.mark.gpu

ODD_SIZES = [1, 3, 4, 5, 127, 1024, 4097, 12289, 70001]


@pytest.mark.parametrize("opt,dt", [(configs.SGD, configs.F32), (configs.ADAM, configs.F32),
                                    (configs.SGD, configs.BF16), (configs.ADAM, configs.BF16)])
@pytest.mark.parametrize("W", [1, 2, 5, 8, 33, 70])
@pytest.mark.parametrize("kernel", [1, 2, 3], ids=["ldg", "bulk", "inline"])
def test_odd_sizes_bit_exact(opt, dt, W, kernel):
    # W = 70 with fp32 gradients exceeds what one ring stage can hold, so the
    # bulk-copy kernel hands those chunks to its direct-load path.
    cfg = tiny_config(ODD_SIZES, W, opt=opt, grad_dtype=dt)
    pair = Pair(cfg, kernel=kernel)
    try:
        every = configs.rounds_all(cfg)[0]
        for it in range(3):
            pair.push_iteration(it)
            pair.aggregate(every)
            pair.compare()
    finally:
        pair.close()


@pytest.mark.parametrize("chunk", [1024, 2048, 8192, 65536])
@pytest.mark.parametrize("kernel", [1, 2, 3], ids=["ldg", "bulk", "inline"])
def test_chunk_size_and_order_invariance(chunk, kernel):
    cfg = tiny_config([5, 40000, 1024, 300001, 77], 4)
    pair = Pair(cfg, kernel=kernel)
    try:
        pair.svc.set_option(B.PS_OPT_CHUNK_ELEMS, chunk)
        pair.svc.set_option(B.PS_OPT_SORT_TASKS, chunk % 2048 == 0)
        order = [(0, 3), (0, 0), (0, 4), (0, 1), (0, 2)]
        for it in range(2):
            pair.push_iteration(it)
            pair.aggregate(order)
        pair.compare()
    finally:
        pair.close()


@pytest.mark.parametrize("kernel", [1, 2, 3], ids=["ldg", "bulk", "inline"])
def test_unaligned_shards_take_scalar_path_same_bits(kernel):
    cfg = tiny_config([4099, 600], 3)
    pair = Pair(cfg, kernel=kernel)
    try:
        job = cfg.jobs[0]
        slab = generate.grad_slab(cfg, 0, 0)
        host = to_np(slab)
        # device copy shifted by one float: every shard pointer is only 4-byte aligned
        dbuf = torch.empty(slab.numel() + 1, dtype=torch.float32, device="cuda")
        dbuf[1:].copy_(slab.reshape(-1))
        base = dbuf.data_ptr() + 4
        for b in job.blocks:
            for w in range(3):
                off = w * job.num_params + b.job_offset
                pair.svc.push(0, b.block, w, base + 4 * off)
                pair.ora.push(0, b.block, w, host[w, b.job_offset:b.job_offset + b.nelem])
        plan = pair.svc.plan([(0, 0), (0, 1)])
        assert any(c.vector_path == 0 for c in plan)
        pair.aggregate([(0, 0), (0, 1)])
        pair.compare()
        with pytest.raises(B.PsError) as e:
            pair.svc.push(0, 0, 0, base + 2)
        assert e.value.status == B.PS_ERR_ALIGN
    finally:
        pair.close()


@pytest.mark.parametrize("kernel", [1, 2, 3], ids=["ldg", "bulk", "inline"])
def test_c1_ten_iterations(kernel):
    cfg = configs.c1()
    pair = Pair(cfg, kernel=kernel)
    try:
        every = configs.rounds_all(cfg)[0]
        for it in range(cfg.iterations):
            pair.push_iteration(it)
            pair.aggregate(every)
            if it in (0, cfg.iterations - 1):
                pair.compare()
    finally:
        pair.close()


@pytest.mark.parametrize("opt", [configs.SGD, configs.ADAM])
def test_bf16_every_bit_pattern_sums_like_the_oracle(opt):
    """The vector path adds bf16 shards with a widening add instruction; the
    oracle widens (bits << 16) and adds in binary32.  Every one of the 65,536
    bf16 patterns meets finite, subnormal, huge and infinite partners here."""
    reps, W = 4, 3
    n = 65536 * reps
    cfg = tiny_config([n], W, opt=opt, grad_dtype=configs.BF16, weight_decay=0.0)
    pair = Pair(cfg)
    try:
        rng = np.random.default_rng(77)
        every = np.tile(np.arange(65536, dtype=np.uint16), reps)
        partner = rng.integers(0, 65536, n, dtype=np.uint16)
        partner[:65536] &= 0x807F                      # subnormal or zero partners for the first copy
        partner[65536:2 * 65536] = (partner[65536:2 * 65536] & 0x80FF) | 0x3A00   # around 1e-3
        third = rng.integers(0, 65536, n, dtype=np.uint16)
        third[2 * 65536:3 * 65536] = 0x0001            # the smallest subnormal
        shards = [partner, every, third]
        dev = []
        for w, a in enumerate(shards):
            t = torch.from_numpy(a.view(np.int16).copy()).view(torch.bfloat16).cuda()
            dev.append(t)
            pair.svc.push(0, 0, w, t)
            pair.ora.push(0, 0, w, a)
        pair.aggregate([(0, 0)])
        p, a, v, _ = pair.gpu_block(0, 0)
        rp = pair.ora.pull(0, 0)
        ra, rv = pair.ora.state(0, 0)
        for got, ref in ((p, rp), (a, ra)) + (((v, rv),) if rv is not None else ()):
            nan = np.isnan(ref)
            assert np.array_equal(np.isnan(got), nan)
            assert np.array_equal(got[~nan].view(np.uint32), ref[~nan].view(np.uint32))
        assert (~np.isnan(ra)).sum() > n // 2
    finally:
        pair.close()


@pytest.mark.parametrize("opt", [configs.SGD, configs.ADAM])
@pytest.mark.parametrize("kernel", [1, 2, 3], ids=["ldg", "bulk", "inline"])
@pytest.mark.parametrize("shift", [0, 1], ids=["vector", "scalar"])
def test_fp32_special_values_travel_like_ieee_binary32(opt, kernel, shift):
    """No flush to zero, no fast division or root, no special cases: gradients
    drawn from ALL binary32 bit patterns (subnormals, huge values that overflow
    the sum, infinities, NaNs, sums that cancel to a signed zero) leave the
    same bits in p and the state as the oracle's plain IEEE arithmetic, over
    two iterations (the second consumes the state the first one left).  NaN
    payloads are not compared: where the oracle has a NaN the kernel has one."""
    W, n = 3, (1 << 18) + 37
    # (no weight decay: wd * p would bury a subnormal aggregate, and with it a flushed one)
    cfg = tiny_config([n], W, opt=opt, weight_decay=0.0)
    pair = Pair(cfg, kernel=kernel)
    try:
        rng = np.random.default_rng(2204)
        q = n // 4
        s0 = rng.integers(0, 1 << 32, n, dtype=np.uint64).astype(np.uint32)
        s1 = rng.integers(0, 1 << 32, n, dtype=np.uint64).astype(np.uint32)
        s1[:q] &= 0x807FFFFF                                   # subnormal or zero
        s1[q:2 * q] = (s1[q:2 * q] & 0x807FFFFF) | 0x7F000000  # about 1e38: sums overflow
        s1[2 * q:3 * q] = s0[2 * q:3 * q] ^ 0x80000000         # the negative of worker 0: cancels
        s1[3 * q::3] = 0x7F800000                              # +inf
        s1[3 * q + 1::3] = 0xFF800000                          # -inf
        s2 = rng.integers(0, 1 << 23, n, dtype=np.uint64).astype(np.uint32)    # positive subnormals
        s2[1::2] |= 0x80000000
        s2[2 * q:3 * q:2] = 0                                  # +0 after a cancelled sum
        shards = [s0.view(np.float32), s1.view(np.float32), s2.view(np.float32)]
        keep = []
        for w, a in enumerate(shards):
            buf = torch.empty(n + 4, dtype=torch.float32, device="cuda")
            buf[shift:shift + n].copy_(torch.from_numpy(a.copy()))
            keep.append(buf)
        for it in range(2):
            for w, a in enumerate(shards):
                pair.svc.push(0, 0, w, keep[w].data_ptr() + 4 * shift)
                pair.ora.push(0, 0, w, a)
            if it == 0:
                assert all(c.vector_path == (0 if shift else 1) for c in pair.svc.plan([(0, 0)]))
            pair.aggregate([(0, 0)])
            p, a, v, _ = pair.gpu_block(0, 0)
            rp = pair.ora.pull(0, 0)
            ra, rv = pair.ora.state(0, 0)
            for name, got, ref in (("p", p, rp), ("state0", a, ra)) + ((("state1", v, rv),) if rv is not None else ()):
                nan = np.isnan(ref)
                assert np.array_equal(np.isnan(got), nan), "%s, iteration %d: NaN positions" % (name, it + 1)
                assert np.array_equal(got[~nan].view(np.uint32), ref[~nan].view(np.uint32)), \
                    "%s, iteration %d: bits" % (name, it + 1)
            # the case has teeth: the state holds NaNs, infinities and non-zero subnormals
            tiny = np.finfo(np.float32).tiny
            assert np.isfinite(ra).sum() > n // 3 and np.isnan(ra).any() and (it > 0 or np.isinf(ra).any())
            assert ((ra != 0) & (np.abs(ra) < tiny)).sum() > 100
    finally:
        pair.close()


@pytest.mark.parametrize("kernel", [1, 2, 3], ids=["ldg", "bulk", "inline"])
@pytest.mark.parametrize("dt", [configs.F32, configs.BF16])
def test_the_sum_follows_worker_order_not_arrival_order(kernel, dt):
    """g0 = 2^24, g1 = g2 = 1 (all exact in bf16 too): in worker order the ones are rounded
    away one at a time and G = 2^24; summed as they ARRIVE (2, 1, 0) G would be 2^24 + 2."""
    n = 12289
    cfg = tiny_config([n], 3, grad_dtype=dt, lr=1.0, momentum=0.0, weight_decay=0.0)
    pair = Pair(cfg, kernel=kernel)
    try:
        vals = {0: 2.0 ** 24, 1: 1.0, 2: 1.0}
        keep = []
        for w in (2, 1, 0):
            t = torch.full((n,), vals[w], dtype=torch.float32, device="cuda")
            host = np.full(n, vals[w], np.float32)
            if dt == configs.BF16:
                t = t.to(torch.bfloat16)
                host = (host.view(np.uint32) >> 16).astype(np.uint16)
            keep.append(t)
            pair.svc.push(0, 0, w, t)
            pair.ora.push(0, 0, w, host)
        pair.aggregate([(0, 0)])
        p, v, _, _ = pair.gpu_block(0, 0)
        assert np.array_equal(v, pair.ora.state(0, 0)[0]) and np.array_equal(p, pair.ora.pull(0, 0))
        assert float(v[0]) == float(v[-1]) == 2.0 ** 24
    finally:
        pair.close()


def test_small_rounds_travel_as_kernel_parameters_and_slots_stay_clean():
    """A round whose table fits the kernel-parameter limit launches without an
    upload.  Tasks of several chunks count their chunks in per-slot device
    state that the finalizing CTA clears: twenty rounds reuse every slot, and
    the per-block norm (summed by the finalizer) must be right every time."""
    cfg = tiny_config([40000, 5, 70001, 1024], 4, opt=configs.ADAM)
    pair = Pair(cfg, kernel=3)
    try:
        pair.svc.set_option(B.PS_OPT_PROFILE, 1)
        every = configs.rounds_all(cfg)[0]
        for it in range(20):
            pair.push_iteration(it % 3)
            if it == 0:
                assert len(pair.svc.plan(every)) > 8      # several chunks per task
            pair.aggregate(every if it % 2 else every[::-1])
            assert pair.svc.launch_info()["kernel"] == "inline"
            if it % 5 == 4 or it < 2:
                pair.compare()
                for b in range(4):
                    busy, span = pair.svc.block_profile(0, b)
                    assert 0.0 < busy < 1e5 and 0.0 < span < 1e5
        # a table too large for the parameter space is uploaded as before
        big = tiny_config([300] * 40, 4)
        other = Pair(big, kernel=3)
        try:
            other.push_iteration(0)
            other.aggregate(configs.rounds_all(big)[0])
            assert other.svc.launch_info()["kernel"] == "ldg"
            other.compare()
        finally:
            other.close()
    finally:
        pair.close()


def test_results_repeat_bit_for_bit_across_runs():
    outs = []
    for _ in range(2):
        cfg = tiny_config([100003, 4096, 17], 8, opt=configs.ADAM, grad_dtype=configs.BF16)
        pair = Pair(cfg)
        try:
            for it in range(2):
                pair.push_iteration(it)
                pair.aggregate(configs.rounds_all(cfg)[0])
            outs.append([pair.gpu_block(0, b)[:3] for b in range(3)] + [pair.svc.block_stats(0, 0)])
        finally:
            pair.close()
    for x, y in zip(outs[0][:3], outs[1][:3]):
        for a, b in zip(x, y):
            assert np.array_equal(a, b)
    assert outs[0][3] == outs[1][3]      # the norm is reduced in a fixed order


def test_bsp_bookkeeping_and_errors_on_device():
    cfg = tiny_config([1000, 2000], 2)
    pair = Pair(cfg)
    svc = pair.svc
    try:
        g = torch.zeros(2000, device="cuda")
        svc.push(0, 0, 0, g)
        with pytest.raises(B.PsError) as e:
            svc.aggregate([(0, 0)])
        assert e.value.status == B.PS_ERR_NOT_READY
        with pytest.raises(B.PsError) as e:
            svc.push(0, 0, 0, g)
        assert e.value.status == B.PS_ERR_DUPLICATE
        svc.push(0, 0, 1, g)
        with pytest.raises(B.PsError) as e:
            svc.aggregate([(0, 0), (0, 0)])
        assert e.value.status == B.PS_ERR_DUPLICATE
        with pytest.raises(B.PsError) as e:
            svc.aggregate([(0, 0), (0, 1)])
        assert e.value.status == B.PS_ERR_NOT_READY
        assert svc.block_stats(0, 0) == (0.0, 0)
        before = svc.launch_info()["launches"]
        svc.aggregate([])
        assert svc.launch_info()["launches"] == before
        svc.aggregate([(0, 0)])
        assert svc.block_stats(0, 0) == (0.0, 1)
        assert svc.launch_info()["launches"] == before + 1
        with pytest.raises(B.PsError) as e:
            svc.aggregate([(0, 0)])          # pushes were consumed
        assert e.value.status == B.PS_ERR_NOT_READY
    finally:
        pair.close()


def test_sqnorm_all_ones_and_host_push_pull():
    cfg = tiny_config([50000], 2, lr=0.5, momentum=0.0, weight_decay=0.0)
    pair = Pair(cfg)
    svc = pair.svc
    try:
        ones = torch.ones(50000).pin_memory()
        s = torch.cuda.Stream()
        svc.push_host(0, 0, 0, ones, s)
        svc.push_host(0, 0, 1, ones, s)
        svc.aggregate([(0, 0)], s)
        out = torch.empty(50000).pin_memory()
        svc.pull_host(0, 0, out, s)
        s.synchronize()
        sq, step = svc.block_stats(0, 0)
        assert sq == 4.0 * 50000 and step == 1
        p0 = generate.init_params(cfg, 0)
        assert torch.equal(out, p0 - 0.5 * 2.0)
    finally:
        pair.close()


@pytest.mark.parametrize("opt,dt", [(configs.SGD, configs.F32), (configs.ADAM, configs.BF16)])
def test_pinned_host_shards_are_read_in_place(opt, dt):
    """Pinned host memory is addressable from the device: ps_push takes the
    pinned pointer and the kernel reads the shard over PCIe, no staging copy."""
    cfg = tiny_config([70001, 4096, 33], 3, opt=opt, grad_dtype=dt)
    pair = Pair(cfg)
    try:
        job = cfg.jobs[0]
        every = configs.rounds_all(cfg)[0]
        for it in range(2):
            slab = generate.grad_slab(cfg, 0, it)
            pinned = generate.empty_slab(slab.shape[0], slab.shape[1], slab.dtype, "cpu")
            base = pinned._base.pin_memory()                     # same padded row layout, page-locked
            pinned = base[:, :slab.shape[1]]
            pinned.copy_(slab)
            host = to_np(slab)
            for b in job.blocks:
                for w in range(job.num_workers):
                    pair.svc.push(0, b.block, w, generate.shard_ptr(pinned, w, b.job_offset))
                    pair.ora.push(0, b.block, w, host[w, b.job_offset:b.job_offset + b.nelem])
            pair.aggregate(every)
            torch.cuda.synchronize()                             # the pinned buffer is released after this
        pair.compare()
    finally:
        pair.close()


@pytest.mark.parametrize("opt,dt", [(configs.SGD, configs.F32), (configs.ADAM, configs.BF16)])
@pytest.mark.parametrize("layout", ["packed", "scattered"])
def test_batched_pushes_from_host_memory(opt, dt, layout):
    """ps_push_host_batch: shards in pinned host memory, either in the layout the
    library sends as one copy (block after block, worker after worker, rows
    padded to 256 bytes) or anywhere; three iterations reuse the staging region
    while the previous aggregate may still be reading it; a block registered
    after the region was allocated gets staging of its own."""
    sizes = [70_001, 5, 4096, 12_345, 300_000]
    cfg = tiny_config(sizes, 3, opt=opt, grad_dtype=dt)
    pair = Pair(cfg)
    svc = pair.svc
    try:
        job = cfg.jobs[0]
        esz = 2 if dt == configs.BF16 else 4
        rows = [(b.nelem * esz + 255) // 256 * 256 for b in job.blocks]
        total = sum(r * job.num_workers for r in rows)
        stream = torch.cuda.Stream()
        every = configs.rounds_all(cfg)[0]
        pools = []
        for it in range(3):
            slab = generate.grad_slab(cfg, 0, it)
            host = to_np(slab)
            raw = slab.contiguous().view(torch.uint8) if dt == configs.F32 else slab.contiguous().view(torch.int16).view(torch.uint8)
            pool = torch.zeros(2 * total + 4096, dtype=torch.uint8).pin_memory()
            pools.append(pool)                                   # stays alive until the copies have run
            jobs, blocks, workers, ptrs = [], [], [], []
            cur = 0
            for b, row in zip(job.blocks, rows):
                for w in range(job.num_workers):
                    off = cur if layout == "packed" else 2 * total - cur - row + (16 if b.block % 2 else 0)
                    n = b.nelem * esz
                    pool[off:off + n].copy_(raw[w, b.job_offset * esz:b.job_offset * esz + n])
                    jobs.append(0); blocks.append(b.block); workers.append(w); ptrs.append(pool.data_ptr() + off)
                    pair.ora.push(0, b.block, w, host[w, b.job_offset:b.job_offset + b.nelem])
                    cur += row
            svc.push_host_batch(np.array(jobs, np.int32), np.array(blocks, np.int32), np.array(workers, np.int32),
                                np.array(ptrs, np.uint64), stream)
            pair.aggregate(every, stream)
        # a (block, worker) twice in one batch, and a batch with one bad entry, change nothing
        one = np.array([0], np.int32)
        with pytest.raises(B.PsError) as e:
            svc.push_host_batch(np.array([0, 0], np.int32), np.array([1, 1], np.int32), np.array([2, 2], np.int32),
                                np.array([pools[0].data_ptr()] * 2, np.uint64), stream)
        assert e.value.status == B.PS_ERR_DUPLICATE
        with pytest.raises(B.PsError) as e:
            svc.push_host_batch(np.array([0, 0], np.int32), np.array([1, 9], np.int32), np.array([0, 0], np.int32),
                                np.array([pools[0].data_ptr()] * 2, np.uint64), stream)
        assert e.value.status == B.PS_ERR_BAD_ARG
        with pytest.raises(B.PsError) as e:
            svc.aggregate([(0, 1)], stream)
        assert e.value.status == B.PS_ERR_NOT_READY
        # a block that did not exist when the job's staging region was laid out
        late = torch.full((1000,), 0.25).pin_memory()
        svc.register_block(0, 7, 1000, 0, None)
        pair.ora.register_block(0, 7, 1000, 0, None)
        ldata = late.to(torch.bfloat16) if dt == configs.BF16 else late
        for w in range(job.num_workers):
            svc.push_host_batch(one, np.array([7], np.int32), np.array([w], np.int32),
                                np.array([ldata.data_ptr()], np.uint64), stream)
            pair.ora.push(0, 7, w, to_np(ldata))
        pair.aggregate([(0, 7)], stream)
        stream.synchronize()
        pair.compare()
        n = 1000
        assert np.array_equal(svc.view(svc.pull(0, 7), n).cpu().numpy(), pair.ora.pull(0, 7))
    finally:
        pair.close()
