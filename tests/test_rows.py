"""Row-sparse push: the oracle's definition (dense with +0.0 rows), host-side
validation of ps_push_rows (CPU), and CUDA parity (GPU)."""
import numpy as np
import pytest
import torch

from oracle import aggregator as A
from paper_2204_03211_b200 import binding as B, build


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def _status(fn, *a):
    try:
        fn(*a)
    except B.PsError as e:
        return e.status
    return 0


# ------------------------------------------------------------------ oracle pin (CPU)

def test_oracle_sparse_push_is_the_dense_push_with_zero_rows_including_signed_zero():
    rows, L, W = 6, 4, 3
    hp = A.HParams(opt=A.SGD, num_workers=W, lr=1.0, momentum=0.0, weight_decay=0.0)
    neg0 = np.float32(-0.0)
    vals = {0: np.array([[1, 2, 3, 4], [neg0, neg0, 5, neg0]], np.float32),         # rows 1, 4
            1: np.array([[neg0, neg0, neg0, neg0]], np.float32),                    # row 4
            2: np.zeros((0, L), np.float32)}
    ids = {0: [1, 4], 1: [4], 2: []}
    o = A.OracleAggregator()
    j = o.register_job(hp)
    o.register_block(j, 0, rows * L)
    for w in range(W):
        o.push_rows(j, 0, w, ids[w], L, vals[w])
    o.aggregate([(j, 0)])
    v = o.state(j, 0)[0].reshape(rows, L)          # v' = G with mom = 0
    assert np.array_equal(v[1], [1, 2, 3, 4]) and not v[[0, 2, 3, 5]].any()
    # row 4: (-0 + -0) + 0 = +0 in columns 0,1,3 (worker 2 is absent); column 2 = 5
    assert np.array_equal(v[4], [0, 0, 5, 0]) and not np.signbit(v[4]).any()
    with pytest.raises(ValueError):
        o.push_rows(j, 0, 0, [3, 2], L, np.zeros((2, L), np.float32))      # not increasing


# ------------------------------------------------------------------ host logic (CPU)

def test_push_rows_validation_and_plan_on_a_planning_only_service():
    s = B.Service(B.PS_DEVICE_NONE, 1, 1 << 30)
    j = s.register_job(num_workers=2)
    big = s.register_job(num_workers=33)
    s.register_block(j, 0, 400 * 100)
    s.register_block(j, 1, 1001)
    s.register_block(big, 0, 400)
    ids, vals = 4096, 8192
    assert _status(s.push_rows, j, 0, 0, ids, 3, 0, vals) == B.PS_ERR_BAD_ARG          # row_len
    assert _status(s.push_rows, j, 0, 0, ids, 101, 400, vals) == B.PS_ERR_BAD_ARG      # more rows than the block has
    assert _status(s.push_rows, j, 1, 0, ids, 1, 400, vals) == B.PS_ERR_BAD_ARG        # 1001 is not whole rows
    assert _status(s.push_rows, j, 0, 0, 0, 3, 400, vals) == B.PS_ERR_BAD_ARG          # NULL ids
    assert _status(s.push_rows, j, 0, 0, ids, 3, 402, vals) == B.PS_ERR_BAD_ARG        # 40000 % 402
    assert _status(s.push_rows, j, 0, 0, ids, 3, 50, vals) == B.PS_ERR_ALIGN           # 200-byte rows
    assert _status(s.push_rows, j, 0, 0, ids, 3, 400, vals + 4) == B.PS_ERR_ALIGN
    assert _status(s.push_rows, big, 0, 0, ids, 1, 400, vals) == B.PS_ERR_BAD_ARG      # W > 32
    s.push_rows(j, 0, 0, ids, 3, 400, vals)
    assert _status(s.push_rows, j, 0, 0, ids, 3, 400, vals) == B.PS_ERR_DUPLICATE
    assert _status(s.push_rows, j, 0, 1, ids, 3, 200, vals) == B.PS_ERR_BAD_ARG        # another row_len
    assert _status(s.plan, [(j, 0)]) == B.PS_ERR_NOT_READY
    s.push(j, 0, 1, 12288)                                                             # dense push from worker 1
    plan = s.plan([(j, 0)])
    assert sum(c.elem_count for c in plan) == 40000
    assert all(c.elem_begin % 400 == 0 and c.elem_count % 400 == 0 for c in plan)      # chunks are whole rows
    assert max(c.elem_count for c in plan) <= (4 * 8192 // 400) * 400      # at most 4x the dense chunk size


# ------------------------------------------------------------------ CUDA parity (GPU)

def _sparse_case(opt, dt, W, rows, L, frac, seed, mixed):
    rng = np.random.default_rng(seed)
    gdt = torch.bfloat16 if dt == B.PS_BF16 else torch.float32
    kw = dict(opt=opt, grad_dtype=dt, num_workers=W, lr=0.1 if opt == B.PS_SGD else 1e-3, momentum=0.9,
              weight_decay=1e-2)
    svc = B.Service(0, 1, 256 << 20)
    ora = A.OracleAggregator()
    j = svc.register_job(**kw)
    assert ora.register_job(A.HParams(**kw)) == j
    init = rng.normal(0, 0.05, size=rows * L).astype(np.float32)
    svc.register_block(j, 0, rows * L, 0, init)
    ora.register_block(j, 0, rows * L, 0, init)
    keep = []
    for it in range(3):
        for w in range(W):
            dense = torch.from_numpy(rng.normal(0, 1e-2, size=(rows, L)).astype(np.float32))
            if it == 1:
                dense[::7] = -0.0                               # rows of negative zeros
            mask = torch.from_numpy(rng.random(rows) < frac)
            if w == 1 and it == 2:
                mask[:] = False                                 # a worker with no rows at all
            dense = (dense * mask[:, None]).to(gdt)
            if mixed and w == 0:
                d = dense.cuda()
                keep.append(d)
                svc.push(j, 0, w, d)
                host = d.cpu()
                ora.push(j, 0, w, (host.view(torch.int16).numpy().view(np.uint16) if gdt == torch.bfloat16
                                   else host.numpy()).reshape(-1))
                continue
            ids = mask.nonzero().squeeze(1).to(torch.int32)
            vals = dense[ids.long()].contiguous()
            if ids.numel() == 0:
                vals = torch.zeros((1, L), dtype=gdt)           # a valid pointer, zero rows
            di, dv = ids.cuda() if ids.numel() else torch.zeros(1, dtype=torch.int32, device="cuda"), vals.cuda()
            keep += [di, dv]
            svc.push_rows(j, 0, w, di, int(ids.numel()), L, dv)
            hv = vals[:ids.numel()]
            ora.push_rows(j, 0, w, ids.numpy(), L,
                          hv.view(torch.int16).numpy().view(np.uint16) if gdt == torch.bfloat16 else hv.numpy())
        svc.aggregate([(j, 0)])
        ora.aggregate([(j, 0)])
        torch.cuda.synchronize()
        s0, s1, _ = svc.block_state(j, 0)
        n = rows * L
        assert np.array_equal(svc.view(svc.pull(j, 0), n).cpu().numpy(), ora.pull(j, 0)), "params, iteration %d" % it
        got_s0 = svc.view(s0, n).cpu().numpy()
        assert np.array_equal(got_s0.view(np.uint32), ora.state(j, 0)[0].view(np.uint32)), "state0 bits (signed zeros too)"
        if s1:
            assert np.array_equal(svc.view(s1, n).cpu().numpy(), ora.state(j, 0)[1])
        sq, step = svc.block_stats(j, 0)
        rsq, rstep = ora.block_stats(j, 0)
        assert step == rstep == it + 1 and abs(sq - rsq) <= 1e-5 * abs(rsq) + 1e-300
    assert svc.device_status() == 0
    svc.close()


@pytest.mark.gpu
@pytest.mark.parametrize("opt,dt", [(B.PS_SGD, B.PS_F32), (B.PS_ADAM, B.PS_F32), (B.PS_SGD, B.PS_BF16),
                                    (B.PS_ADAM, B.PS_BF16)])
@pytest.mark.parametrize("W,rows,L,frac,mixed", [(1, 50, 8, 0.3, False), (4, 2621, 400, 0.05, False),
                                                 (8, 333, 400, 0.05, True), (32, 100, 64, 0.5, False),
                                                 (3, 41, 1000, 0.0, False)])
def test_row_sparse_push_equals_dense_semantics_bit_for_bit(opt, dt, W, rows, L, frac, mixed):
    _sparse_case(opt, dt, W, rows, L, frac, seed=W * 1000 + rows, mixed=mixed)
