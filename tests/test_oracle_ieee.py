"""Pins the oracle's binary32 arithmetic at the edges of the format.

The GPU parity test on special values compares the kernels with the oracle on
gradients drawn from all bit patterns; that proves something only if the
oracle itself neither flushes subnormals nor special-cases anything.  Every
expected value here is a bit pattern worked out by hand from IEEE-754
(round to nearest even, gradual underflow), for inputs chosen so that the
exact result is representable or its rounding is obvious.
"""
from fractions import Fraction

import numpy as np
import pytest

from oracle import aggregator as A


def bits(*words):
    return np.array(words, dtype=np.uint32).view(np.float32)


def as_bits(a):
    return [int(x) for x in np.asarray(a, dtype=np.float32).view(np.uint32)]


def nearest_f32(q: Fraction) -> np.float32:
    """The binary32 value nearest to the exact rational q (ties do not occur in the uses here)."""
    c = np.float32(float(q))
    cands = [c, np.nextafter(c, np.float32(np.inf)), np.nextafter(c, np.float32(-np.inf))]
    dist = [abs(Fraction(float(x)) - q) for x in cands]
    assert sorted(dist)[0] != sorted(dist)[1]
    return cands[dist.index(min(dist))]


def sgd(W, lr=1.0, momentum=0.0, wd=0.0):
    return A.HParams(opt=A.SGD, num_workers=W, lr=lr, momentum=momentum, weight_decay=wd)


def step(hp, shards, p0, t=1, s0=None, s1=None):
    p = np.array(p0, dtype=np.float32)
    s0 = np.zeros_like(p) if s0 is None else np.array(s0, dtype=np.float32)
    if hp.opt == A.ADAM:
        s1 = np.zeros_like(p) if s1 is None else np.array(s1, dtype=np.float32)
    with np.errstate(all="ignore"):
        sq = A.block_step(hp, t, [np.ascontiguousarray(g, dtype=np.float32) for g in shards], p, s0, s1)
    return p, s0, s1, sq


@pytest.mark.parametrize("W", [1, 2, 3, 7, 32])
def test_subnormal_shards_add_up_exactly(W):
    # W copies of the smallest subnormal (bits 1) sum to bits W; with lr = 1 and p0 = 0
    # the parameter is its negative.  A flush to zero anywhere gives +-0 instead.
    g = bits(1, 1, 0x80000001)
    p, v, _, _ = step(sgd(W), [g] * W, [0.0, 0.0, 0.0])
    assert as_bits(v) == [W, W, 0x80000000 | W]
    assert as_bits(p) == [0x80000000 | W, 0x80000000 | W, W]


def test_subnormal_plus_subnormal_crosses_into_the_normal_range():
    # 0x007FFFFF (largest subnormal) + 0x00000001 = 0x00800000 (smallest normal), exactly
    p, v, _, _ = step(sgd(2), [bits(0x007FFFFF), bits(0x00000001)], [0.0])
    assert as_bits(v) == [0x00800000]


def test_product_that_underflows_is_rounded_not_flushed():
    # lr * v' with lr = 0.5 and v' = 3 * 2^-149: 1.5 * 2^-149 is a tie between bits 1 and 2, even wins
    p, v, _, _ = step(sgd(1, lr=0.5), [bits(3)], [0.0])
    assert as_bits(v) == [3] and as_bits(p) == [0x80000002]
    # momentum 0.5 on a state of 2^-149 (bits 1): 0.5 * 2^-149 is a tie between 0 and bits 1: +0
    p, v, _, _ = step(sgd(1, lr=1.0, momentum=0.5), [bits(0)], [0.0], s0=bits(1))
    assert as_bits(v) == [0] and as_bits(p) == [0]


def test_sum_overflows_to_infinity_and_opposite_infinities_give_nan():
    big = bits(0x7F7FFFFF)                                         # the largest finite value
    p, v, _, sq = step(sgd(2), [np.repeat(big, 2), np.repeat(big, 2)], [1.0, -1.0])
    assert as_bits(v) == [0x7F800000] * 2 and as_bits(p) == [0xFF800000] * 2
    assert np.isinf(sq)
    p, v, _, _ = step(sgd(2), [bits(0x7F800000), bits(0xFF800000)], [1.0])
    assert np.isnan(v[0]) and np.isnan(p[0])
    # an infinity survives a finite partner and the order of the workers does not matter for it
    p, v, _, _ = step(sgd(3), [bits(0x3F800000), bits(0xFF800000), bits(0x7F7FFFFF)], [0.0])
    assert as_bits(v) == [0xFF800000] and as_bits(p) == [0x7F800000]


def test_cancelled_sum_is_plus_zero_and_signed_zeros_follow_the_rules():
    x = bits(0x3FC00000, 0xC2F6E979)                               # 1.5, -123.456
    # x + (-x) = +0 under round to nearest; v' = +0; p' = p - lr * (+0) keeps p, also p = -0
    p, v, _, _ = step(sgd(2), [x, -x], bits(0x80000000, 0x40490FDB))
    assert as_bits(v) == [0, 0]
    assert as_bits(p) == [0x80000000, 0x40490FDB]
    # G = (-0) + (-0) = -0, but d = G + wd * p = (-0) + (+0) = +0 with p = +0: v' = +0, p' = +0
    p, v, _, _ = step(sgd(2), [bits(0x80000000), bits(0x80000000)], [0.0])
    assert as_bits(v) == [0] and as_bits(p) == [0]
    # every term -0 (p = -0, state -0): d = (-0) + (0 * -0) = -0, v' = (0 * -0) + (-0) = -0,
    # p' = (-0) - (1 * -0) = (-0) + (+0) = +0
    p, v, _, _ = step(sgd(2), [bits(0x80000000), bits(0x80000000)], bits(0x80000000), s0=bits(0x80000000))
    assert as_bits(v) == [0x80000000] and as_bits(p) == [0]


def test_nan_in_one_worker_reaches_parameter_and_state_only_at_its_own_element():
    g0 = bits(0x3F800000, 0x7FC00000, 0x3F800000)
    g1 = bits(0x3F800000, 0x3F800000, 0x3F800000)
    p, v, _, sq = step(sgd(2), [g0, g1], [0.0, 0.0, 0.0])
    assert as_bits(v)[0] == as_bits(v)[2] == 0x40000000 and np.isnan(v[1])
    assert as_bits(p)[0] == as_bits(p)[2] == 0xC0000000 and np.isnan(p[1])
    assert np.isnan(sq)


def test_adam_with_subnormal_gradient_keeps_gradual_underflow():
    # b1 = 0.5: m' = 0.5 * d exactly.  d = 2^-148 (bits 2) gives m' = 2^-149 (bits 1).
    # d * d underflows to +0, v' = 0, den = sqrt(0) / sbc2 + eps = eps; the step is
    # ss_1 * (m' / eps) with ss_1 = lr / (1 - b1) = 2 lr.
    hp = A.HParams(opt=A.ADAM, num_workers=1, lr=0.25, beta1=0.5, beta2=0.999, eps=1e-8)
    p, m, v, _ = step(hp, [bits(2)], [0.0])
    assert as_bits(m) == [1] and as_bits(v) == [0]
    quo = nearest_f32(Fraction(1, 2 ** 149) / Fraction(float(np.float32(1e-8))))   # one correctly rounded division
    want = -np.float32(np.float32(0.5) * quo)                          # ss_1 = 0.25 / 0.5 = 0.5, exact scaling
    assert as_bits(p) == as_bits([want])
    assert 0 < abs(float(p[0])) and np.isfinite(p[0])


def test_adam_root_and_quotient_are_correctly_rounded():
    # v' = omb2 * d^2 with b2 = 0.75 (omb2 = 0.25, exact) and d = 3: v' = 2.25, sqrt = 1.5 exactly;
    # t = 1: sbc2 = sqrt(1 - 0.75) = 0.5, so sqrt(v') / sbc2 = 3; eps = 1 gives den = 4.
    # b1 = 0.5: m' = 1.5, ss_1 = lr / 0.5; lr = 0.5 gives ss_1 = 1: p' = p0 - 1.5 / 4 = p0 - 0.375.
    hp = A.HParams(opt=A.ADAM, num_workers=1, lr=0.5, beta1=0.5, beta2=0.75, eps=1.0)
    p, m, v, _ = step(hp, [np.float32([3.0, -3.0])], [1.0, 1.0])
    assert list(m) == [1.5, -1.5] and list(v) == [2.25, 2.25]
    assert list(p) == [0.625, 1.375]
    # a quotient that is not representable: m' / den = 0.5 / 3 must be the nearest binary32 to 1/6.
    # d = 1, b1 = 0.5 -> m' = 0.5; b2 = 0.75 -> v' = 0.25, sqrt = 0.5, / 0.5 = 1, + eps 2 = 3.
    hp = A.HParams(opt=A.ADAM, num_workers=1, lr=0.5, beta1=0.5, beta2=0.75, eps=2.0)
    p, m, v, _ = step(hp, [np.float32([1.0])], [0.0])
    assert as_bits(p) == as_bits([-np.float32(1.0 / 6.0)]) == [0xBE2AAAAB]
