"""Pins the CPU oracle to closed forms, hand-worked values and invariants.

The paper prints no worked aggregation example (Section 2 only says that the
server updates the master copy with the aggregated result), so the oracle is
pinned to what the mathematics fixes.  Each pin is chosen so that a plausible
mistake (dropped term, wrong sign, wrong operand, wrong worker order) fails.
Expected values here are computed by hand or by Python/numpy binary64
arithmetic written independently of the oracle's source.
"""
import math
import os

import numpy as np
import pytest

from oracle import aggregator as A

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _table(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                rows.append([float(x) for x in line.split()])
    return rows


def f32(x):
    return np.asarray(x, dtype=np.float32)


# ------------------------------------------------------------------ reduce

@pytest.mark.parametrize("W", [1, 2, 3, 4, 8, 16, 32])
def test_identical_shards_sum_to_W_times_g(W):
    # g = small integers * 2^-10: the running sums k*g stay exactly
    # representable, so the closed form W*g must hold bit for bit.
    rng = np.random.default_rng(W)
    g = f32(rng.integers(-2048, 2048, size=257) * 2.0 ** -10)
    hp = A.HParams(opt=A.SGD, num_workers=W, lr=1.0, momentum=0.0, weight_decay=0.0)
    p, v = np.zeros(257, np.float32), np.zeros(257, np.float32)
    sq = A.block_step(hp, 1, [g] * W, p, v)
    assert np.array_equal(v, f32(W) * g)          # v' = 0*v + G
    assert np.array_equal(p, -(f32(W) * g))       # p' = 0 - 1*G
    assert sq == float(np.sum((np.float64(W) * g.astype(np.float64)) ** 2))


def test_identical_shards_arbitrary_values_within_ulps():
    rng = np.random.default_rng(5)
    W = 16
    g = f32(rng.normal(0, 1e-2, size=1000))
    hp = A.HParams(opt=A.SGD, num_workers=W, lr=1.0)
    p, v = np.zeros(1000, np.float32), np.zeros(1000, np.float32)
    A.block_step(hp, 1, [g] * W, p, v)
    exact = W * g.astype(np.float64)
    assert np.all(np.abs(v - exact) <= (W - 1) * np.spacing(np.abs(f32(exact))))


def test_single_worker_passes_gradient_through_bit_for_bit():
    g = f32(np.random.default_rng(1).normal(0, 1, size=100))
    hp = A.HParams(opt=A.SGD, num_workers=1, lr=1.0)
    p, v = np.zeros(100, np.float32), np.zeros(100, np.float32)
    A.block_step(hp, 1, [g], p, v)
    assert np.array_equal(v, g) and np.array_equal(p, -g)


def test_distinct_integer_shards_sum_exactly():
    W, n = 8, 64
    shards = [f32(np.arange(n) * (w + 1) - 7 * w) for w in range(W)]
    hp = A.HParams(opt=A.SGD, num_workers=W, lr=1.0)
    p, v = np.zeros(n, np.float32), np.zeros(n, np.float32)
    A.block_step(hp, 1, shards, p, v)
    assert np.array_equal(v, f32(sum(s.astype(np.int64) for s in shards)))


def test_worker_order_is_0_to_W_minus_1():
    # (2^24 + 1) + (-2^24): the first add rounds to 2^24 (ties-to-even), so the
    # fixed order 0,1,2 gives 0 while the order 0,2,1 gives exactly 1.
    a, b, c = f32([2.0 ** 24]), f32([1.0]), f32([-(2.0 ** 24)])
    hp = A.HParams(opt=A.SGD, num_workers=3, lr=1.0)
    p, v = np.zeros(1, np.float32), np.zeros(1, np.float32)
    A.block_step(hp, 1, [a, b, c], p, v)
    assert v[0] == 0.0
    p, v = np.zeros(1, np.float32), np.zeros(1, np.float32)
    A.block_step(hp, 1, [a, c, b], p, v)
    assert v[0] == 1.0


def test_sum_not_mean_and_grad_scale():
    g = f32([0.5, -1.5])
    hp = A.HParams(opt=A.SGD, num_workers=4, lr=1.0, grad_scale=0.25)
    p, v = np.zeros(2, np.float32), np.zeros(2, np.float32)
    sq = A.block_step(hp, 1, [g] * 4, p, v)
    assert np.array_equal(v, g)                   # (4 g) * 0.25
    assert sq == 0.25 + 2.25                      # norm of the SCALED aggregate


# ------------------------------------------------------------------ SGD

def test_zero_gradient_zero_decay_leaves_parameters_fixed():
    rng = np.random.default_rng(2)
    p0 = f32(rng.normal(0, 0.05, size=333))
    p, v = p0.copy(), np.zeros(333, np.float32)
    hp = A.HParams(opt=A.SGD, num_workers=4, lr=0.1, momentum=0.9, weight_decay=0.0)
    z = np.zeros(333, np.float32)
    for t in range(1, 6):
        assert A.block_step(hp, t, [z] * 4, p, v) == 0.0
    assert np.array_equal(p, p0) and not v.any()


def test_momentum_recurrence_by_hand():
    hp = A.HParams(opt=A.SGD, num_workers=2, lr=0.25, momentum=0.5, weight_decay=0.0)
    p, v = np.zeros(5, np.float32), np.zeros(5, np.float32)
    g = np.full(5, 0.5, np.float32)
    for t, ev, ep in _table("momentum_recurrence.txt"):
        A.block_step(hp, int(t), [g, g], p, v)
        assert np.all(v == np.float32(ev)) and np.all(p == np.float32(ep))


def test_weight_decay_recurrence_by_hand():
    z = np.zeros(3, np.float32)
    hp0 = A.HParams(opt=A.SGD, num_workers=1, lr=0.5, momentum=0.0, weight_decay=0.5)
    hp5 = A.HParams(opt=A.SGD, num_workers=1, lr=0.5, momentum=0.5, weight_decay=0.5)
    pa, va = np.full(3, 1024, np.float32), z.copy()
    pb, vb = np.full(3, 1024, np.float32), z.copy()
    for t, p_nomom, v_mom, p_mom in _table("weight_decay_recurrence.txt"):
        A.block_step(hp0, int(t), [z], pa, va)
        A.block_step(hp5, int(t), [z], pb, vb)
        assert np.all(pa == np.float32(p_nomom))
        assert np.all(vb == np.float32(v_mom)) and np.all(pb == np.float32(p_mom))


@pytest.mark.parametrize("mu,lr", [(0.9, 0.1), (0.5, 0.01), (0.0, 0.3)])
def test_sgd_constant_gradient_closed_form(mu, lr):
    # v_t = G (1 - mu^t)/(1 - mu);  p_t = p_0 - lr * sum_{k<=t} v_k
    W, G = 4, 0.0123
    g = np.full(7, G / W, np.float32)
    Gf = float(np.float32(G / W)) * W
    hp = A.HParams(opt=A.SGD, num_workers=W, lr=lr, momentum=mu, weight_decay=0.0)
    p, v = np.full(7, 0.3, np.float32), np.zeros(7, np.float32)
    mu32, lr32 = float(np.float32(mu)), float(np.float32(lr))
    acc = 0.0
    for t in range(1, 21):
        A.block_step(hp, t, [g] * W, p, v)
        vt = Gf * (1 - mu32 ** t) / (1 - mu32) if mu32 != 1 else Gf * t
        acc += vt
        assert np.allclose(v, vt, rtol=1e-6, atol=0)
        assert np.allclose(p, float(np.float32(0.3)) - lr32 * acc, rtol=0, atol=1e-6)


def test_weight_decay_geometric_closed_form():
    # G = 0, mom = 0:  p_t = p_0 (1 - lr*wd)^t
    lr, wd = np.float32(0.1), np.float32(1e-2)
    hp = A.HParams(opt=A.SGD, num_workers=2, lr=float(lr), momentum=0.0, weight_decay=float(wd))
    p0 = f32(np.linspace(-1, 1, 11))
    p, v = p0.copy(), np.zeros(11, np.float32)
    z = np.zeros(11, np.float32)
    for t in range(1, 31):
        A.block_step(hp, t, [z, z], p, v)
        want = p0.astype(np.float64) * (1 - float(lr) * float(wd)) ** t
        assert np.allclose(p, want, rtol=1e-6, atol=1e-9)


def test_weight_decay_enters_with_plus_sign_and_uses_old_p():
    # one step, mom = 0: p' = p - lr*(G + wd*p)
    hp = A.HParams(opt=A.SGD, num_workers=1, lr=0.5, momentum=0.0, weight_decay=0.25)
    p, v = f32([8.0, -8.0]), np.zeros(2, np.float32)
    A.block_step(hp, 1, [f32([1.0, 1.0])], p, v)
    assert np.array_equal(v, f32([3.0, -1.0]))
    assert np.array_equal(p, f32([6.5, -7.5]))


# ------------------------------------------------------------------ Adam

def test_adam_by_hand_three_steps():
    hp = A.HParams(opt=A.ADAM, num_workers=1, lr=0.5, beta1=0.5, beta2=0.75, eps=0.0)
    p, m, v = (np.zeros(4, np.float32) for _ in range(3))
    g = np.full(4, 2.0, np.float32)
    for t, em, ev, ep in _table("adam_first_steps.txt"):
        A.block_step(hp, int(t), [g], p, m, v)
        assert np.all(m == np.float32(em)) and np.all(v == np.float32(ev))
        assert np.allclose(p, ep, rtol=0, atol=2e-7)


def test_adam_first_step_closed_form():
    # from zero state, wd = 0:  p_1 = p_0 - lr * g / (|g| + eps)
    rng = np.random.default_rng(3)
    g = f32(rng.normal(0, 1e-3, size=500))
    p0 = f32(rng.normal(0, 0.05, size=500))
    lr, eps = 1e-4, 1e-8
    hp = A.HParams(opt=A.ADAM, num_workers=2, lr=lr, beta1=0.9, beta2=0.999, eps=eps)
    p, m, v = p0.copy(), np.zeros(500, np.float32), np.zeros(500, np.float32)
    A.block_step(hp, 1, [g, np.zeros(500, np.float32)], p, m, v)
    G = g.astype(np.float64)
    want = p0 - float(np.float32(lr)) * G / (np.abs(G) + float(np.float32(eps)))
    assert np.max(np.abs(p - want)) <= 1e-6 * (1 + np.max(np.abs(want)))
    assert np.allclose(m, (1 - float(np.float32(0.9))) * G, rtol=1e-6)
    assert np.allclose(v, (1 - float(np.float32(0.999))) * G * G, rtol=1e-5)


def test_adam_constant_gradient_closed_form():
    # constant g: mhat = g, vhat = g^2 at every t  =>  p_t = p_0 - t*lr*g/(|g|+eps)
    g = f32([3e-3, -7e-4, 1e-2, -2.5e-1])
    lr, eps = 1e-3, 1e-8
    hp = A.HParams(opt=A.ADAM, num_workers=1, lr=lr, beta1=0.9, beta2=0.999, eps=eps)
    p, m, v = np.zeros(4, np.float32), np.zeros(4, np.float32), np.zeros(4, np.float32)
    G = g.astype(np.float64)
    for t in range(1, 41):
        A.block_step(hp, t, [g], p, m, v)
        want = -t * float(np.float32(lr)) * G / (np.abs(G) + float(np.float32(eps)))
        assert np.max(np.abs(p - want)) <= 1e-6 * (1 + np.max(np.abs(want))) + 2e-7 * t


def test_adam_eps_sits_outside_the_root_and_decay_is_coupled():
    # v' = (1-b2) d^2 with d = G + wd*p;  den = sqrt(v')/sqrt(1-b2) + eps = |d| + eps
    hp = A.HParams(opt=A.ADAM, num_workers=1, lr=1.0, beta1=0.0, beta2=0.75, eps=1.0, weight_decay=0.5)
    p, m, v = f32([2.0]), np.zeros(1, np.float32), np.zeros(1, np.float32)
    A.block_step(hp, 1, [f32([1.0])], p, m, v)      # d = 2, m = 2, v = 1, den = 2/1 + 1 = 3
    assert m[0] == 2.0 and v[0] == 1.0
    assert abs(float(p[0]) - (2.0 - 2.0 / 3.0)) < 2e-7


def test_adam_bias_scalars():
    lib = A.lib()
    for t in (1, 2, 10, 1000):
        assert lib.oracle_adam_step_size(np.float32(1e-4), np.float32(0.9), t) == \
            float(np.float32(1e-4)) / (1.0 - float(np.float32(0.9)) ** t)
        assert lib.oracle_adam_sqrt_bc2(np.float32(0.999), t) == \
            math.sqrt(1.0 - float(np.float32(0.999)) ** t)


# ------------------------------------------------------------------ bf16

def test_bf16_widening_exhaustive():
    bits = np.arange(65536, dtype=np.uint32)
    want = (bits << 16).astype(np.uint32).view(np.float32)
    got = A.widen_bf16(bits.astype(np.uint16))
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


def test_bf16_shards_equal_widened_f32_shards():
    rng = np.random.default_rng(4)
    W, n = 5, 300
    bits = [rng.integers(0x3000, 0x3f00, size=n).astype(np.uint16) | (rng.integers(0, 2, size=n).astype(np.uint16) << 15)
            for _ in range(W)]
    wide = [(b.astype(np.uint32) << 16).view(np.float32) for b in bits]
    kw = dict(opt=A.ADAM, num_workers=W, lr=1e-3)
    pa, ma, va = (np.zeros(n, np.float32) for _ in range(3))
    pb, mb, vb = (np.zeros(n, np.float32) for _ in range(3))
    sa = A.block_step(A.HParams(grad_dtype=A.BF16, **kw), 1, bits, pa, ma, va)
    sb = A.block_step(A.HParams(grad_dtype=A.F32, **kw), 1, wide, pb, mb, vb)
    assert sa == sb and np.array_equal(pa, pb) and np.array_equal(ma, mb) and np.array_equal(va, vb)


# ------------------------------------------------------------------ f32 vs f64, stats

@pytest.mark.parametrize("opt", [A.SGD, A.ADAM])
def test_f32_mode_tracks_f64_truth(opt):
    rng = np.random.default_rng(6)
    W, n, T = 8, 4096, 20
    hp = A.HParams(opt=opt, num_workers=W, lr=0.1 if opt == A.SGD else 1e-3, momentum=0.9, weight_decay=1e-4)
    p0 = rng.normal(0, 0.05, size=n).astype(np.float32)
    p32, a32, b32 = p0.copy(), np.zeros(n, np.float32), np.zeros(n, np.float32)
    p64, a64, b64 = p0.astype(np.float64), np.zeros(n), np.zeros(n)
    for t in range(1, T + 1):
        shards = [rng.normal(0, 1e-3, size=n).astype(np.float32) for _ in range(W)]
        s32 = A.block_step(hp, t, shards, p32, a32, b32, mode="f32")
        s64 = A.block_step(hp, t, shards, p64, a64, b64, mode="f64")
        assert abs(s32 - s64) <= 1e-5 * s64
    tol = 1e-6 if opt == A.SGD else 2e-5       # Adam's m/sqrt(v) amplifies rounding of tiny v
    assert np.max(np.abs(p32 - p64) / (1 + np.abs(p64))) <= tol
    assert np.max(np.abs(a32 - a64)) <= 1e-6 * (1 + np.max(np.abs(a64)))


def test_sqnorm_of_all_ones_block_is_nelem():
    n = 12345
    hp = A.HParams(opt=A.SGD, num_workers=1, lr=0.0)
    sq = A.block_step(hp, 1, [np.ones(n, np.float32)], np.zeros(n, np.float32), np.zeros(n, np.float32))
    assert sq == float(n)


# ------------------------------------------------------------------ service semantics

def _mk(num_contexts=1):
    o = A.OracleAggregator(num_contexts=num_contexts, nthreads=2)
    j = o.register_job(A.HParams(opt=A.SGD, num_workers=2, lr=0.1, momentum=0.9, weight_decay=1e-4))
    return o, j


def test_blocks_are_independent_and_order_free():
    rng = np.random.default_rng(7)
    sizes = [5, 1000, 33, 4097]
    init = [f32(rng.normal(0, 0.05, size=n)) for n in sizes]
    grads = [[[f32(rng.normal(0, 1e-2, size=n)) for _ in range(2)] for n in sizes] for _ in range(3)]
    results = []
    for order in ([0, 1, 2, 3], [3, 1, 0, 2]):
        o, j = _mk()
        for b, n in enumerate(sizes):
            o.register_block(j, b, n, init=init[b])
        for it in range(3):
            for b in order:
                for w in range(2):
                    o.push(j, b, w, grads[it][b][w])
            o.aggregate([(j, b) for b in order])
        results.append([o.pull(j, b).copy() for b in range(4)])
    for a, b in zip(*results):
        assert np.array_equal(a, b)
    # a block aggregated alone equals the same block aggregated in a pack
    o, j = _mk()
    o.register_block(j, 0, sizes[1], init=init[1])
    for it in range(3):
        for w in range(2):
            o.push(j, 0, w, grads[it][1][w])
        o.aggregate([(j, 0)])
    assert np.array_equal(o.pull(j, 0), results[0][1])


def test_bsp_rules_not_ready_duplicate_push_duplicate_task():
    o, j = _mk()
    o.register_block(j, 0, 4)
    g = np.ones(4, np.float32)
    o.push(j, 0, 0, g)
    with pytest.raises(RuntimeError):
        o.aggregate([(j, 0)])                  # only 1 of 2 workers pushed
    with pytest.raises(ValueError):
        o.push(j, 0, 0, g)                     # one request per task per iteration
    o.push(j, 0, 1, g)
    with pytest.raises(ValueError):
        o.aggregate([(j, 0), (j, 0)])
    assert o.block_stats(j, 0)[1] == 0         # rejected calls changed nothing
    o.aggregate([(j, 0)])
    assert o.block_stats(j, 0) == (4 * 4.0, 1)
    with pytest.raises(RuntimeError):
        o.aggregate([(j, 0)])                  # pushes were consumed


def test_migration_preserves_the_version():
    rng = np.random.default_rng(8)
    n = 777
    init = f32(rng.normal(0, 0.05, size=n))
    grads = [[f32(rng.normal(0, 1e-2, size=n)) for _ in range(2)] for _ in range(6)]
    outs = []
    for migrate in (False, True):
        o, j = _mk(num_contexts=2)
        o.register_block(j, 0, n, ctx=0, init=init)
        for it in range(6):
            if migrate and it in (2, 4):
                o.migrate_block(j, 0, 1 - o.blocks[(j, 0)].ctx)
            for w in range(2):
                o.push(j, 0, w, grads[it][w])
            o.aggregate([(j, 0)])
        outs.append((o.pull(j, 0).copy(), o.state(j, 0)[0].copy(), o.block_stats(j, 0)[1]))
    assert np.array_equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][1], outs[1][1])
    assert outs[0][2] == outs[1][2] == 6
