"""Pins of the oracle's SERVICE semantics (oracle/aggregator.py, the Python
layer above the plain C++ loops): who is summed in which order, what a
row-sparse push stands for, what migration keeps, where the state starts,
what the per-block norm covers.  Each expected value is worked out by hand.

These were written after planting mistakes in a copy of that layer
(tests/test_oracle_mutants.py) showed which of them no pin noticed.
"""
import numpy as np
import pytest

from oracle import aggregator as A


def bits(a):
    return [int(x) for x in np.asarray(a, np.float32).view(np.uint32)]


def service(W, opt=A.SGD, contexts=1, **kw):
    o = A.OracleAggregator(contexts)
    hp = dict(opt=opt, num_workers=W, lr=1.0, momentum=0.0, weight_decay=0.0)
    hp.update(kw)
    assert o.register_job(A.HParams(**hp)) == 0
    return o


def test_shards_are_summed_in_worker_order_whatever_the_arrival_order():
    # g0 = 2^24, g1 = g2 = 1.  Worker order: (2^24 + 1) rounds back to 2^24, twice: G = 2^24.
    # Arrival order 1, 2, 0 would give (1 + 1) + 2^24 = 2^24 + 2.
    g = {0: np.float32([2.0 ** 24]), 1: np.float32([1.0]), 2: np.float32([1.0])}
    for arrival in ([0, 1, 2], [1, 2, 0], [2, 1, 0]):
        o = service(3)
        o.register_block(0, 0, 1, 0, [0.0])
        for w in arrival:
            o.push(0, 0, w, g[w])
        o.aggregate([(0, 0)])
        assert float(o.state(0, 0)[0][0]) == 2.0 ** 24, arrival         # v' = G
        assert float(o.pull(0, 0)[0]) == -(2.0 ** 24), arrival


def test_state_starts_at_zero_and_the_first_aggregate_is_step_one():
    # momentum 0.5, first step from zero state: v' = 0.5 * 0 + g = g exactly
    o = service(1, momentum=0.5)
    o.register_block(0, 0, 3, 0, [1.0, 2.0, 3.0])
    o.push(0, 0, 0, np.float32([0.25, -0.5, 4.0]))
    o.aggregate([(0, 0)])
    assert list(o.state(0, 0)[0]) == [0.25, -0.5, 4.0]
    assert list(o.pull(0, 0)) == [0.75, 2.5, -1.0]
    assert o.block_stats(0, 0)[1] == 1
    # Adam: both moments start at zero — m' = (1 - b1) g, v' = (1 - b2) g^2 with b1 = b2 = 0.5
    a = service(1, opt=A.ADAM, lr=0.5, beta1=0.5, beta2=0.5, eps=1.0)
    a.register_block(0, 0, 1, 0, [0.0])
    a.push(0, 0, 0, np.float32([2.0]))
    a.aggregate([(0, 0)])
    m, v = a.state(0, 0)
    assert float(m[0]) == 1.0 and float(v[0]) == 2.0


def test_the_norm_is_that_of_the_last_aggregate_only():
    o = service(2)
    o.register_block(0, 0, 4, 0, None)
    for it, val in enumerate([1.0, 3.0]):
        for w in range(2):
            o.push(0, 0, w, np.full(4, val, np.float32))
        o.aggregate([(0, 0)])
        sq, step = o.block_stats(0, 0)
        assert step == it + 1 and sq == 4 * (2 * val) ** 2                # sum over 4 elements of (2 val)^2


def test_rows_a_sparse_push_leaves_out_count_as_plus_zero():
    """Iteration 1 makes the momentum negative and keeps p negative; in iteration 2
    (momentum coefficient 0, decay coefficient 0) v' = (0 * v) + (G + 0 * p) = (-0) + (G + (-0)).
    Worker 0 sends a dense -0.0 for row 1, worker 1 a row-sparse shard without row 1:
    G = (-0) + (+0) = +0, so v' = +0.  Were the missing row -0.0, G and v' would be -0.0."""
    o = service(2, lr=2.0 ** -10)
    o.register_block(0, 0, 4, 0, [-10.0] * 4)                             # two rows of two
    for w in range(2):
        o.push(0, 0, w, np.float32([-1.0, -1.0, -1.0, -1.0]))
    o.aggregate([(0, 0)])
    assert list(o.state(0, 0)[0]) == [-2.0] * 4 and all(p < 0 for p in o.pull(0, 0))
    neg0 = np.float32(-0.0)
    o.push(0, 0, 0, np.array([0.5, 0.5, neg0, neg0], np.float32))         # dense, row 1 = -0.0
    o.push_rows(0, 0, 1, [0], 2, np.float32([[0.25, 0.25]]))              # row 0 only
    o.aggregate([(0, 0)])
    assert bits(o.state(0, 0)[0]) == bits([0.75, 0.75, 0.0, 0.0])         # +0.0, not -0.0, in row 1


def test_row_ids_must_be_strictly_increasing_and_in_range():
    o = service(1)
    o.register_block(0, 0, 6, 0, None)                                    # three rows of two
    row = np.float32([[1.0, 1.0], [2.0, 2.0]])
    for bad in ([1, 1], [2, 0], [0, 3], [-1, 0]):
        with pytest.raises(ValueError):
            o.push_rows(0, 0, 0, bad, 2, row)
    with pytest.raises(ValueError):
        o.push_rows(0, 0, 0, [0], 4, np.float32([[1.0] * 4]))             # 6 elements are not whole rows of 4
    o.push_rows(0, 0, 0, [0, 2], 2, row)
    o.aggregate([(0, 0)])
    assert list(o.state(0, 0)[0]) == [1.0, 1.0, 0.0, 0.0, 2.0, 2.0]


def test_migration_moves_the_block_to_the_named_context_with_everything_it_holds():
    o = service(1, contexts=3, momentum=0.5)
    o.register_block(0, 0, 2, 1, [1.0, 1.0])
    o.push(0, 0, 0, np.float32([1.0, 2.0]))
    o.aggregate([(0, 0)])
    assert o.blocks[(0, 0)].ctx == 1
    o.migrate_block(0, 0, 2)
    assert o.blocks[(0, 0)].ctx == 2
    assert o.block_stats(0, 0)[1] == 1                                    # the version travels
    assert list(o.state(0, 0)[0]) == [1.0, 2.0] and list(o.pull(0, 0)) == [0.0, -1.0]
    o.push(0, 0, 0, np.float32([1.0, 2.0]))
    o.aggregate([(0, 0)])                                                 # v' = 0.5 v + g: the state came along
    assert list(o.state(0, 0)[0]) == [1.5, 3.0] and o.block_stats(0, 0)[1] == 2
    with pytest.raises(ValueError):
        o.migrate_block(0, 0, 3)


def test_array_widening_of_bf16_covers_every_element():
    # 0x3F80 = 1.0, 0x4000 = 2.0, 0xC040 = -3.0, 0x0001 = 2^-133 (a bf16 subnormal): the last one too
    got = A.widen_bf16(np.array([0x3F80, 0x4000, 0xC040, 0x0001], np.uint16))
    assert bits(got) == [0x3F800000, 0x40000000, 0xC0400000, 0x00010000]
    assert A.widen_bf16(np.array([0xC040], np.uint16)).tolist() == [-3.0]
