"""The entry point that allocates nothing, checked against the regular one.

ps_aggregate_block_noalloc exists for callers that cannot allocate device
memory at the time of the call — a process whose framework already owns all of
the GPU's memory, or a loop that cannot afford the device-wide stall an
allocation may bring — so its scratch lives in a fixed array inside the
library.  Here the same block is aggregated twice in a row (steps 1 and 2)
through a ps_service and through the no-allocation call, on identical inputs;
parameters and optimizer state must agree bit for bit (both run the same
kernel) and the gradient norm within the tolerance the other tests use.  The
CPU oracle is the second, independent checker of the same two calls.

The file name sorts last on purpose: a run that stops at the first failure has
already been through every other test.  It also passes on its own in a fresh
process, where its first call is the one that looks the scratch address up.
"""
import numpy as np
import pytest
import torch

from oracle import aggregator as A
from paper_2204_03211_b200 import binding as B

pytestmark = pytest.mark.gpu


def _desc(opt, dtype, W):
    if opt == B.PS_ADAM:
        return B.ps_job_desc(opt, dtype, W, 1e-3, 0.0, 1e-2, 0.9, 0.999, 1e-8, 1.0)
    return B.ps_job_desc(opt, dtype, W, 0.1, 0.9, 1e-4, 0.9, 0.999, 1e-8, 1.0)


@pytest.mark.parametrize("opt,dtype,W,nelem", [
    (B.PS_SGD, B.PS_F32, 4, 300_001),        # several chunks and a ragged tail
    (B.PS_ADAM, B.PS_BF16, 3, 70_003),
    (B.PS_SGD, B.PS_F32, 1, 5),              # smaller than one vector
])
def test_no_alloc_entry_matches_service_two_calls_in_a_row(opt, dtype, W, nelem):
    torch.cuda.set_device(0)
    gen = torch.Generator(device="cuda").manual_seed(1234 + nelem)
    gdt = torch.bfloat16 if dtype == B.PS_BF16 else torch.float32
    p0 = torch.randn(nelem, device="cuda", generator=gen) * 0.05
    d = _desc(opt, dtype, W)

    svc = B.Service(0, 1, 64 << 20)
    try:
        j = svc.register_job(opt, dtype, W, d.lr, d.momentum, d.weight_decay, d.beta1, d.beta2, d.eps, d.grad_scale)
        svc.register_block(j, 0, nelem, 0, p0)
        # caller-owned state for the no-allocation call (the TEST may allocate; the entry point may not)
        p = p0.clone()
        s0 = torch.zeros(nelem, device="cuda")
        s1 = torch.zeros(nelem, device="cuda") if opt == B.PS_ADAM else None
        sq = torch.full((1,), -1.0, device="cuda", dtype=torch.float64)
        stream = torch.cuda.Stream()
        torch.cuda.synchronize()
        # the oracle's copy of the same block
        hp = A.HParams(opt, dtype, W, d.lr, d.momentum, d.weight_decay, d.beta1, d.beta2, d.eps, d.grad_scale)
        op = p0.cpu().numpy().copy()
        o0 = np.zeros(nelem, np.float32)
        o1 = np.zeros(nelem, np.float32) if opt == B.PS_ADAM else None
        for step in (1, 2):
            shards = [(torch.randn(nelem, device="cuda", generator=gen) * 1e-2).to(gdt) for _ in range(W)]
            torch.cuda.synchronize()
            host = [g.view(torch.int16).cpu().numpy().view(np.uint16) if dtype == B.PS_BF16 else g.cpu().numpy()
                    for g in shards]
            osq = A.block_step(hp, step, host, op, o0, o1)
            for w, g in enumerate(shards):
                svc.push(j, 0, w, g)
            svc.aggregate([(j, 0)], stream)
            B.ps_aggregate_block_noalloc(d, step, nelem, p, s0, s1, shards, sq, stream)
            stream.synchronize()
            a0, a1, _ = svc.block_state(j, 0)
            ref_p = svc.view(svc.pull(j, 0), nelem)
            assert torch.equal(p, ref_p), "parameters differ at step %d" % step
            assert torch.equal(s0, svc.view(a0, nelem))
            if s1 is not None:
                assert torch.equal(s1, svc.view(a1, nelem))
            ref_sq, ref_step = svc.block_stats(j, 0)
            assert ref_step == step
            assert abs(sq.item() - ref_sq) <= 1e-5 * abs(ref_sq)
            # and against the oracle
            assert np.array_equal(p.cpu().numpy(), op), "parameters differ from the oracle at step %d" % step
            assert np.array_equal(s0.cpu().numpy(), o0)
            if s1 is not None:
                assert np.array_equal(s1.cpu().numpy(), o1)
            assert abs(sq.item() - osq) <= 1e-5 * abs(osq)
    finally:
        svc.close()


def test_norm_output_needs_only_eight_byte_alignment():
    """The norm is one double written by one thread: an output that is 8- but
    not 16-byte aligned (element 1 of a double tensor) is accepted and does not
    change the result (nor push the block onto the scalar path)."""
    torch.cuda.set_device(0)
    nelem, W = 200_000, 4
    gen = torch.Generator(device="cuda").manual_seed(99)
    d = _desc(B.PS_SGD, B.PS_F32, W)
    p0 = torch.randn(nelem, device="cuda", generator=gen) * 0.05
    shards = [torch.randn(nelem, device="cuda", generator=gen) * 1e-2 for _ in range(W)]
    out = torch.full((4,), -1.0, device="cuda", dtype=torch.float64)
    assert out.data_ptr() % 16 == 0
    results = []
    for k in (0, 1):                       # 16-byte aligned, then 8-byte aligned only
        p, s0 = p0.clone(), torch.zeros(nelem, device="cuda")
        torch.cuda.synchronize()
        B.ps_aggregate_block_noalloc(d, 1, nelem, p, s0, None, shards, out.data_ptr() + 8 * k)
        torch.cuda.synchronize()
        results.append((p.cpu().numpy(), s0.cpu().numpy(), float(out[k])))
    assert np.array_equal(results[0][0], results[1][0]) and np.array_equal(results[0][1], results[1][1])
    assert results[0][2] == results[1][2] > 0
    hp = A.HParams(B.PS_SGD, B.PS_F32, W, d.lr, d.momentum, d.weight_decay, d.beta1, d.beta2, d.eps, d.grad_scale)
    op, o0 = p0.cpu().numpy().copy(), np.zeros(nelem, np.float32)
    osq = A.block_step(hp, 1, [g.cpu().numpy() for g in shards], op, o0)
    assert np.array_equal(results[1][0], op) and np.array_equal(results[1][1], o0)
    assert abs(results[1][2] - osq) <= 1e-5 * osq
    with pytest.raises(ValueError):
        B.ps_aggregate_block_noalloc(d, 1, nelem, p0.clone(), torch.zeros(nelem, device="cuda"), None, shards[:3])


def test_no_alloc_entry_rejects_what_it_cannot_hold():
    torch.cuda.set_device(0)
    d = _desc(B.PS_SGD, B.PS_F32, 2)
    buf = torch.zeros(16, device="cuda")
    shards = [buf, buf]
    with pytest.raises(B.PsError) as e:
        B.ps_aggregate_block_noalloc(d, 1, B.PS_NOALLOC_MAX_ELEMS + 1, buf, buf, None, shards)
    assert e.value.status == B.PS_ERR_TOO_LARGE and "PS_NOALLOC_MAX_ELEMS" in str(e.value)
    with pytest.raises(B.PsError) as e:
        B.ps_aggregate_block_noalloc(d, 0, 16, buf, buf, None, shards)          # steps count from 1
    assert e.value.status == B.PS_ERR_BAD_ARG
    with pytest.raises(B.PsError) as e:
        B.ps_aggregate_block_noalloc(_desc(B.PS_ADAM, B.PS_F32, 2), 1, 16, buf, buf, None, shards)   # Adam needs state1
    assert e.value.status == B.PS_ERR_BAD_ARG
    with pytest.raises(B.PsError) as e:
        B.ps_aggregate_block_noalloc(d, 1, 8, buf, buf, None, [buf, buf.data_ptr() + 2])
    assert e.value.status == B.PS_ERR_ALIGN
