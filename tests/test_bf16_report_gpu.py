"""bf16 gradients against the UNROUNDED draws.

Everywhere else both sides consume the same bf16 bit patterns, which is the
gate (bit equality).  Here the CUDA path is fed the rounded bf16 gradients and
the oracle, in its binary32 mode, the fp32 draws they were rounded from: the
difference is what bf16 transport costs, and it has to stay inside the stated
tolerance of 2e-3 relative.

Reading of "relative": bf16 keeps 8 significant bits, so one rounding moves a
gradient by at most 2^-9 = 1.95e-3 of its magnitude, and the aggregated
gradient G = sum_w g_w by at most 2e-3 * sum_w |g_w| — that bound is asserted
element by element, and the same bound carried through the (linear) first
moment of Adam.  The parameter update of Adam is m / (sqrt(v) + eps), a
normalised quantity: where G is close to zero its sign, and with it the whole
step, can flip under any perturbation, so no element-wise relative bound on
the update exists; its median and its L2-norm-wise error are reported and the
median is asserted.
"""
import numpy as np
import pytest
import torch

from helpers import tiny_config, to_np
from oracle import aggregator as A
from paper_2204_03211_b200 import binding as B
from workload import configs, generate

pytestmark = pytest.mark.gpu

TOL = 2e-3          # the stated tolerance for bf16-gradient inputs
W = 32


def _service(cfg):
    job = cfg.jobs[0]
    svc = B.Service(0, 1, 8 * 4 * job.num_params + (1 << 20))
    assert svc.register_job(**job.hparams()) == 0
    return svc


def test_aggregated_gradient_from_bf16_shards_is_within_2e3_of_the_fp32_sum():
    # SGD with lr 1, no momentum, no decay, p0 = 0: the parameters after one aggregate are -G
    cfg = tiny_config([130_001, 4096, 7], W, grad_dtype=configs.BF16, lr=1.0, momentum=0.0, weight_decay=0.0,
                      grad_std=1e-3)
    job = cfg.jobs[0]
    svc = _service(cfg)
    try:
        slab, full = generate.grad_slab(cfg, 0, 0, keep_fp32=True)
        dslab = generate.to_device(slab, torch.device("cuda", 0))
        hp32 = A.HParams(**dict(job.hparams(), grad_dtype=A.F32))
        f = full.numpy()
        for b in job.blocks:
            svc.register_block(0, b.block, b.nelem, 0, None)
            for w in range(W):
                svc.push(0, b.block, w, generate.shard_ptr(dslab, w, b.job_offset))
        svc.aggregate([(0, b.block) for b in job.blocks])
        torch.cuda.synchronize()
        worst = 0.0
        for b in job.blocks:
            sl = slice(b.job_offset, b.job_offset + b.nelem)
            p = np.zeros(b.nelem, np.float32)
            A.block_step(hp32, 1, [f[w, sl].copy() for w in range(W)], p, np.zeros(b.nelem, np.float32))
            got = svc.view(svc.pull(0, b.block), b.nelem).cpu().numpy()
            mass = np.abs(f[:, sl].astype(np.float64)).sum(axis=0)              # sum_w |g_w|
            err = np.abs(got.astype(np.float64) - p.astype(np.float64))
            assert (err <= TOL * mass).all(), "block %d: %g of sum|g|" % (b.block, float((err / mass).max()))
            worst = max(worst, float((err / mass).max()))
        print("\nbf16 transport, aggregated gradient: max |G_bf16 - G_fp32| / sum_w|g_w| = %.3e (bound %.1e)" % (worst, TOL))
    finally:
        svc.close()


def test_adam_three_iterations_bf16_shards_against_fp32_draws():
    # the hyper-parameters of the BERT-large-shaped configuration, on a subset of its block sizes
    cfg = tiny_config([1 << 20, 4096 * 1024 // 4, 1024, 30522], W, opt=configs.ADAM, grad_dtype=configs.BF16,
                      lr=1e-4, momentum=0.0, weight_decay=0.0, grad_std=1e-3)
    job = cfg.jobs[0]
    svc = _service(cfg)
    dev = torch.device("cuda", 0)
    try:
        hp32 = A.HParams(**dict(job.hparams(), grad_dtype=A.F32))
        p0 = generate.init_params(cfg, 0).numpy()
        n = job.num_params
        rp, rm, rv = p0.copy(), np.zeros(n, np.float32), np.zeros(n, np.float32)
        mass_m = np.zeros(n, np.float64)        # the bound carried through m' = b1*m + (1-b1)*G
        for b in job.blocks:
            svc.register_block(0, b.block, b.nelem, 0, p0[b.job_offset:b.job_offset + b.nelem])
        every = [(0, b.block) for b in job.blocks]
        keep = []
        for it in range(3):
            slab, full = generate.grad_slab(cfg, 0, it, keep_fp32=True)
            dslab = generate.to_device(slab, dev)
            keep.append(dslab)
            for b in job.blocks:
                for w in range(W):
                    svc.push(0, b.block, w, generate.shard_ptr(dslab, w, b.job_offset))
            svc.aggregate(every)
            f = full.numpy()
            mass_m = job.beta1 * mass_m + (1.0 - job.beta1) * np.abs(f.astype(np.float64)).sum(axis=0)
            for b in job.blocks:
                sl = slice(b.job_offset, b.job_offset + b.nelem)
                A.block_step(hp32, it + 1, [f[w, sl].copy() for w in range(W)], rp[sl], rm[sl], rv[sl])
        torch.cuda.synchronize()
        gp, gm = np.empty(n, np.float32), np.empty(n, np.float32)
        for b in job.blocks:
            sl = slice(b.job_offset, b.job_offset + b.nelem)
            gp[sl] = svc.view(svc.pull(0, b.block), b.nelem).cpu().numpy()
            gm[sl] = svc.view(svc.block_state(0, b.block)[0], b.nelem).cpu().numpy()
        # first moment: linear in the gradients, so the transport bound carries through
        err_m = np.abs(gm.astype(np.float64) - rm)
        assert (err_m <= TOL * mass_m + 1e-12).all(), "first moment: %g of the bound" % float((err_m / (TOL * mass_m)).max())
        # the update itself: reported; the median is asserted (see the module docstring)
        du_g, du_r = gp.astype(np.float64) - p0, rp.astype(np.float64) - p0
        rel = np.abs(du_g - du_r) / np.maximum(np.abs(du_r), 1e-30)
        med, l2 = float(np.median(rel)), float(np.linalg.norm(du_g - du_r) / np.linalg.norm(du_r))
        beyond = float((rel > TOL).mean())
        print("\nbf16 transport, Adam, 3 iterations, W=32, %d params: update error median %.2e, L2 %.2e, "
              "share of elements beyond 2e-3: %.3f; first moment max %.2e of its bound"
              % (n, med, l2, beyond, float((err_m / (TOL * mass_m + 1e-300)).max())))
        assert med <= TOL
    finally:
        svc.close()
