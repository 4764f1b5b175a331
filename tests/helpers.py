"""Shared test plumbing: drives the CUDA service and the CPU oracle with the
same seeded inputs and compares them element by element."""
from __future__ import annotations

import numpy as np
import torch

from oracle import aggregator as A
from paper_2204_03211_b200 import binding as B
from workload import configs, generate

TOL = 1e-6      # max |delta| <= TOL * (1 + |ref|) for fp32 state (the stated tolerance; bit equality is expected and asserted too)


def to_np(t: torch.Tensor) -> np.ndarray:
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def oracle_hp(job: configs.JobSpec) -> A.HParams:
    return A.HParams(**job.hparams())


def assert_close(got: np.ndarray, ref: np.ndarray, what: str, tol: float = TOL):
    assert got.shape == ref.shape, what
    err = np.abs(got.astype(np.float64) - ref.astype(np.float64))
    bound = tol * (1.0 + np.abs(ref.astype(np.float64)))
    bad = err > bound
    assert not bad.any(), "%s: %d/%d elements off, max err %.3e at %d" % (
        what, int(bad.sum()), bad.size, float(err.max()), int(err.argmax()))


class Pair:
    """One CUDA service and one oracle fed the same registrations and pushes."""

    def __init__(self, cfg: configs.Config, device: int = 0, arena_bytes: int | None = None, nthreads: int = 0,
                 kernel: int = 0):
        self.cfg = cfg
        self.dev = torch.device("cuda", device)
        need = sum(3 * (4 * b.nelem + 256) for j in cfg.jobs for b in j.blocks) + (1 << 20)
        self.svc = B.Service(device, cfg.num_contexts, arena_bytes or need)
        # kernel: 0 automatic, 1 direct loads with an uploaded table, 2 bulk-copy ring,
        # 3 direct loads with the table passed as a kernel parameter where it fits
        self.svc.set_option(B.PS_OPT_KERNEL, 1 if kernel == 3 else kernel)
        if kernel in (1, 3):
            self.svc.set_option(B.PS_OPT_INLINE_TABLE, int(kernel == 3))
        self.ora = A.OracleAggregator(cfg.num_contexts, nthreads)
        self.keep = []          # gradient tensors of the iteration in flight
        for j, job in enumerate(cfg.jobs):
            jid = self.svc.register_job(**job.hparams())
            assert jid == self.ora.register_job(oracle_hp(job)) == j
            p0 = generate.init_params(cfg, j)
            for b in job.blocks:
                init = p0[b.job_offset:b.job_offset + b.nelem].contiguous()
                ctx = configs.initial_context(cfg, j, b.block)
                self.svc.register_block(j, b.block, b.nelem, ctx, init)
                self.ora.register_block(j, b.block, b.nelem, ctx, init.numpy())

    def close(self):
        self.svc.close()

    def push_iteration(self, it: int, jobs=None):
        """Generates iteration `it`'s gradients on the CPU and pushes every
        block of the given jobs to both sides."""
        self.keep = []
        for j, job in enumerate(self.cfg.jobs):
            if jobs is not None and j not in jobs:
                continue
            slab = generate.grad_slab(self.cfg, j, it)
            dslab = generate.to_device(slab, self.dev)
            self.keep.append((slab, dslab))
            host = to_np(slab)
            esz = dslab.element_size()
            for b in job.blocks:
                for w in range(job.num_workers):
                    self.svc.push(j, b.block, w, generate.shard_ptr(dslab, w, b.job_offset))
                    self.ora.push(j, b.block, w, host[w, b.job_offset:b.job_offset + b.nelem])

    def aggregate(self, ready, stream=None):
        self.svc.aggregate(ready, stream)
        self.ora.aggregate(list(ready))

    def migrate(self, job, block, dst, stream=None):
        self.svc.migrate_block(job, block, dst, stream)
        self.ora.migrate_block(job, block, dst)

    def gpu_block(self, j: int, b: int):
        n = self.cfg.jobs[j].blocks[b].nelem
        s0, s1, ctx = self.svc.block_state(j, b)
        torch.cuda.synchronize(self.dev)
        p = self.svc.view(self.svc.pull(j, b), n).cpu().numpy()
        a = self.svc.view(s0, n).cpu().numpy()
        v = self.svc.view(s1, n).cpu().numpy() if s1 else None
        return p, a, v, ctx

    def check_padding(self, j: int, b: int, nelem: int, sections: int, tag: str):
        """Every section of a block's arena range (parameters, state) is rounded
        up to 256 bytes and zeroed at registration; the kernels may never write
        past the last element, so the bytes between 4*nelem and the end of each
        section are still zero (a short overrun would not show in any other
        comparison)."""
        _, _, sec = self.svc.block_location(j, b)
        pad = (sec - 4 * nelem) // 4
        if pad == 0:
            return
        base = self.svc.pull(j, b)
        for k in range(sections):
            tail = self.svc.view(base + k * sec + 4 * nelem, pad).view(torch.int32)
            assert int(tail.abs().max()) == 0, "%s: bytes after section %d were written" % (tag, k)

    def compare(self, sq_rtol: float = 1e-5, exact: bool = True):
        worst = 0.0
        assert self.svc.device_status() == 0, "a bounded wait expired inside a kernel"
        for j, job in enumerate(self.cfg.jobs):
            for b in job.blocks:
                p, a, v, ctx = self.gpu_block(j, b.block)
                rp = self.ora.pull(j, b.block)
                ra, rv = self.ora.state(j, b.block)
                tag = "%s job %d block %d" % (self.cfg.name, j, b.block)
                assert_close(p, rp, tag + " params")
                assert_close(a, ra, tag + " state0")
                if rv is not None:
                    assert_close(v, rv, tag + " state1")
                if exact:
                    assert np.array_equal(p, rp) and np.array_equal(a, ra), tag + " not bit-identical"
                    if rv is not None:
                        assert np.array_equal(v, rv), tag + " state1 not bit-identical"
                assert ctx == self.ora.blocks[(j, b.block)].ctx, tag + " context"
                sq, step = self.svc.block_stats(j, b.block)
                rsq, rstep = self.ora.block_stats(j, b.block)
                assert step == rstep, tag + " step"
                assert abs(sq - rsq) <= sq_rtol * abs(rsq) + 1e-300, tag + " sqnorm %r vs %r" % (sq, rsq)
                worst = max(worst, float(np.max(np.abs(p.astype(np.float64) - rp))))
                self.check_padding(j, b.block, b.nelem, 3 if rv is not None else 2, tag)
        return worst


def tiny_config(sizes, W, opt=configs.SGD, grad_dtype=configs.F32, seed=123, **kw) -> configs.Config:
    """One job whose blocks have the given element counts."""
    from workload import shapes
    tensors = [shapes.Tensor("t%d" % i, (n,), i) for i, n in enumerate(sizes)]
    blocks = shapes.cut_blocks(tensors, keep_whole=lambda t: True)
    base = dict(lr=0.1, momentum=0.9, weight_decay=1e-4, grad_std=1e-2)
    if opt == configs.ADAM:
        base = dict(lr=1e-3, momentum=0.0, weight_decay=1e-2, grad_std=1e-2)
    base.update(kw)
    job = configs.JobSpec("tiny", "tiny", tensors, blocks, W, opt=opt, grad_dtype=grad_dtype, **base)
    return configs.Config("tiny", seed, 3, [job])


class SampledPair:
    """Full-size configurations: the CUDA service holds every block; the oracle
    follows (a) a seeded sample of positions of EVERY block (block edges, chunk
    boundaries, random interior points) packed into one pseudo-block per job —
    valid because the update is element-wise — and (b) a few whole blocks per
    job, for which the per-block norm is checked too.  Gradients are generated
    on the GPU; the oracle receives copies of exactly those bits."""

    def __init__(self, cfg: configs.Config, per_block: int = 48, full_per_job: int = 4, device: int = 0,
                 full_block_limit: int = 1 << 21):
        self.cfg = cfg
        self.dev = torch.device("cuda", device)
        arena = sum(3 * (4 * b.nelem + 256) for j in cfg.jobs for b in j.blocks) + (64 << 20)
        self.svc = B.Service(device, cfg.num_contexts, arena)
        self.ora = A.OracleAggregator(1, 0)
        self.pos, self.full = [], []
        self.ctx = {}
        for j, job in enumerate(cfg.jobs):
            assert self.svc.register_job(**job.hparams()) == j == self.ora.register_job(oracle_hp(job))
            p0 = generate.init_params(cfg, j, self.dev)
            for b in job.blocks:
                c = configs.initial_context(cfg, j, b.block)
                self.ctx[(j, b.block)] = c
                self.svc.register_block(j, b.block, b.nelem, c, p0[b.job_offset:b.job_offset + b.nelem])
            pos = generate.sample_positions(cfg, j, per_block).to(self.dev)
            self.pos.append(pos)
            self.ora.register_block(j, 0, pos.numel(), 0, p0[pos].cpu().numpy())
            # whole blocks: first, last, the smallest and the largest that is not huge
            cand = [b for b in job.blocks if b.nelem <= full_block_limit]
            pick = {cand[0].block, cand[-1].block, min(cand, key=lambda b: b.nelem).block,
                    max(cand, key=lambda b: b.nelem).block}
            pick = sorted(pick)[:full_per_job]
            self.full.append(pick)
            for k, bid in enumerate(pick):
                b = job.blocks[bid]
                self.ora.register_block(j, 1 + k, b.nelem, 0, p0[b.job_offset:b.job_offset + b.nelem].cpu().numpy())
            del p0
        self.slabs = [None] * len(cfg.jobs)

    def close(self):
        self.svc.close()

    def iteration(self, it: int, rounds, stream=None):
        """Pushes fresh gradients for every block, aggregates round by round."""
        cfg = self.cfg
        for j, job in enumerate(cfg.jobs):
            self.slabs[j] = generate.grad_slab(cfg, j, it, self.dev, out=self.slabs[j])
        torch.cuda.synchronize(self.dev)
        for ready in rounds:
            jobs, blocks, workers, ptrs = [], [], [], []
            for (j, b) in ready:
                job = cfg.jobs[j]
                for w in range(job.num_workers):
                    jobs.append(j); blocks.append(b); workers.append(w)
                    ptrs.append(generate.shard_ptr(self.slabs[j], w, job.blocks[b].job_offset))
            self.svc.push_batch(np.array(jobs, np.int32), np.array(blocks, np.int32), np.array(workers, np.int32),
                                np.array(ptrs, np.uint64))
            self.svc.aggregate(ready, stream)
        # oracle: the same bits, sampled columns and whole blocks
        for j, job in enumerate(cfg.jobs):
            samp = to_np(self.slabs[j][:, self.pos[j]])
            ready = [(j, 0)]
            for w in range(job.num_workers):
                self.ora.push(j, 0, w, samp[w])
            for k, bid in enumerate(self.full[j]):
                b = job.blocks[bid]
                whole = to_np(self.slabs[j][:, b.job_offset:b.job_offset + b.nelem])
                for w in range(job.num_workers):
                    self.ora.push(j, 1 + k, w, whole[w])
                ready.append((j, 1 + k))
            self.ora.aggregate(ready)
        torch.cuda.synchronize(self.dev)

    def migrate(self, plan, stream=None):
        """Moves every listed block to the next context: one batched call per destination."""
        by_dst = {}
        for (j, b) in plan:
            dst = (self.ctx[(j, b)] + 1) % self.cfg.num_contexts
            by_dst.setdefault(dst, []).append((j, b))
            self.ctx[(j, b)] = dst
        for dst, tasks in by_dst.items():
            self.svc.migrate_blocks(tasks, dst, stream)

    def _gather(self, j: int):
        """p, s0, s1 of job j at the sampled positions, from the service's memory."""
        job = self.cfg.jobs[j]
        pos = self.pos[j]
        starts = torch.tensor([b.job_offset for b in job.blocks] + [job.num_params], device=self.dev)
        which = torch.searchsorted(starts, pos, right=True) - 1
        outs = [torch.empty(pos.numel(), device=self.dev) for _ in range(3)]
        has_s1 = False
        for b in job.blocks:
            sel = (which == b.block).nonzero().squeeze(1)
            if sel.numel() == 0:
                continue
            loc = pos[sel] - b.job_offset
            s0, s1, ctx = self.svc.block_state(j, b.block)
            assert ctx == self.ctx[(j, b.block)], "block (%d,%d) in the wrong context" % (j, b.block)
            outs[0][sel] = self.svc.view(self.svc.pull(j, b.block), b.nelem)[loc]
            outs[1][sel] = self.svc.view(s0, b.nelem)[loc]
            if s1:
                has_s1 = True
                outs[2][sel] = self.svc.view(s1, b.nelem)[loc]
        return outs[0].cpu().numpy(), outs[1].cpu().numpy(), outs[2].cpu().numpy() if has_s1 else None

    def compare(self, expect_step: int, sq_rtol: float = 1e-5):
        assert self.svc.device_status() == 0
        torch.cuda.synchronize(self.dev)
        for j, job in enumerate(self.cfg.jobs):
            tag = "%s job %d" % (self.cfg.name, j)
            p, a, v = self._gather(j)
            rp = self.ora.pull(j, 0)
            ra, rv = self.ora.state(j, 0)
            assert_close(p, rp, tag + " sampled params")
            assert_close(a, ra, tag + " sampled state0")
            assert np.array_equal(p, rp) and np.array_equal(a, ra), tag + " samples not bit-identical"
            if rv is not None:
                assert_close(v, rv, tag + " sampled state1")
                assert np.array_equal(v, rv), tag + " sampled state1 not bit-identical"
            for k, bid in enumerate(self.full[j]):
                n = job.blocks[bid].nelem
                got = self.svc.view(self.svc.pull(j, bid), n).cpu().numpy()
                assert np.array_equal(got, self.ora.pull(j, 1 + k)), tag + " whole block %d" % bid
                sq, step = self.svc.block_stats(j, bid)
                rsq, rstep = self.ora.block_stats(j, 1 + k)
                assert step == rstep == expect_step, tag + " step of block %d" % bid
                assert abs(sq - rsq) <= sq_rtol * abs(rsq) + 1e-300, tag + " sqnorm of block %d" % bid
            for b in job.blocks[:: max(1, len(job.blocks) // 16)]:
                assert self.svc.block_stats(j, b.block)[1] == expect_step


class FullPair:
    """Full-size configurations compared IN FULL: the CUDA service and the
    oracle both hold every block; every iteration the gradients are generated
    on the GPU, the service aggregates them round by round, and the oracle
    receives a host copy of exactly those bits, job by job (the largest slab is
    a few GB), and follows every element of every block.  compare() then checks
    every element of parameters and optimizer state bit for bit, every block's
    step counter, context and gradient norm.  Launch configuration = what
    bench.py times (overlapped launches, rounds given with their inputs
    complete, packing over time)."""

    def __init__(self, cfg: configs.Config, device: int = 0, overlap: int = 1, kernel: int = 0):
        self.cfg = cfg
        self.dev = torch.device("cuda", device)
        arena = sum(3 * (4 * b.nelem + 256) for j in cfg.jobs for b in j.blocks) + (64 << 20)
        self.svc = B.Service(device, cfg.num_contexts, arena)
        self.svc.set_option(B.PS_OPT_OVERLAP, overlap)
        if kernel:
            self.svc.set_option(B.PS_OPT_KERNEL, kernel)
        self.ora = A.OracleAggregator(cfg.num_contexts, 0)
        self.ctx = {}
        for j, job in enumerate(cfg.jobs):
            assert self.svc.register_job(**job.hparams()) == j == self.ora.register_job(oracle_hp(job))
            p0 = generate.init_params(cfg, j, self.dev)
            h0 = p0.cpu().numpy()
            for b in job.blocks:
                c = configs.initial_context(cfg, j, b.block)
                self.ctx[(j, b.block)] = c
                self.svc.register_block(j, b.block, b.nelem, c, p0[b.job_offset:b.job_offset + b.nelem])
                self.ora.register_block(j, b.block, b.nelem, c, h0[b.job_offset:b.job_offset + b.nelem])
            del p0, h0
        self.slabs = [None] * len(cfg.jobs)
        self.stream = torch.cuda.Stream(self.dev)

    def close(self):
        self.svc.close()

    def iteration(self, it: int, rounds):
        cfg = self.cfg
        for j in range(len(cfg.jobs)):
            self.slabs[j] = generate.grad_slab(cfg, j, it, self.dev, out=self.slabs[j])
        torch.cuda.synchronize(self.dev)          # the gradients are complete before they are pushed
        for ready in rounds:
            jobs, blocks, workers, ptrs = [], [], [], []
            for (j, b) in ready:
                job = cfg.jobs[j]
                for w in range(job.num_workers):
                    jobs.append(j); blocks.append(b); workers.append(w)
                    ptrs.append(generate.shard_ptr(self.slabs[j], w, job.blocks[b].job_offset))
            self.svc.round(np.array(jobs, np.int32), np.array(blocks, np.int32), np.array(workers, np.int32),
                           np.array(ptrs, np.uint64), ready, B.PS_ROUND_INPUTS_COMPLETE, self.stream)
        self.svc.join(self.stream)
        # the oracle: the same bits, every block, one job's slab on the host at a time
        for j, job in enumerate(cfg.jobs):
            host = to_np(self.slabs[j])
            ready = []
            for b in job.blocks:
                for w in range(job.num_workers):
                    self.ora.push(j, b.block, w, host[w, b.job_offset:b.job_offset + b.nelem])
                ready.append((j, b.block))
            self.ora.aggregate(ready)
            del host
        self.stream.synchronize()

    def migrate(self, plan, stream=None):
        """Moves every listed block to the next context: one batched call per destination."""
        by_dst = {}
        for (j, b) in plan:
            dst = (self.ctx[(j, b)] + 1) % self.cfg.num_contexts
            by_dst.setdefault(dst, []).append((j, b))
            self.ctx[(j, b)] = dst
            self.ora.migrate_block(j, b, dst)
        for dst, tasks in by_dst.items():
            self.svc.migrate_blocks(tasks, dst, stream)

    def compare(self, expect_step: int, sq_rtol: float = 1e-5):
        assert self.svc.device_status() == 0
        torch.cuda.synchronize(self.dev)
        elems = 0
        for j, job in enumerate(self.cfg.jobs):
            for b in job.blocks:
                tag = "%s job %d block %d" % (self.cfg.name, j, b.block)
                s0, s1, ctx = self.svc.block_state(j, b.block)
                assert ctx == self.ctx[(j, b.block)] == self.ora.blocks[(j, b.block)].ctx, tag + " context"
                ra, rv = self.ora.state(j, b.block)
                got = self.svc.view(self.svc.pull(j, b.block), b.nelem).cpu().numpy()
                assert np.array_equal(got, self.ora.pull(j, b.block)), tag + " params not bit-identical"
                assert np.array_equal(self.svc.view(s0, b.nelem).cpu().numpy(), ra), tag + " state0 not bit-identical"
                if rv is not None:
                    assert np.array_equal(self.svc.view(s1, b.nelem).cpu().numpy(), rv), tag + " state1 not bit-identical"
                sq, step = self.svc.block_stats(j, b.block)
                rsq, rstep = self.ora.block_stats(j, b.block)
                assert step == rstep == expect_step, tag + " step"
                assert abs(sq - rsq) <= sq_rtol * abs(rsq) + 1e-300, tag + " sqnorm %r vs %r" % (sq, rsq)
                elems += b.nelem
        assert elems == self.cfg.num_params
        return elems
