"""Are the parity checkers themselves awake?  After an ordinary aggregate that
compares clean, ONE thing is changed on the oracle's side, on the CPU — one
ulp in one element in the middle of a large block, a step counter, a norm by a
few parts in 10^5, a context — and the comparison has to fail.  No kernel is
altered; the one thing written on the GPU is a float in a block's own padding
(inside the arena), by the test, for the check that watches the padding.
"""
import numpy as np
import pytest
import torch

from helpers import FullPair, Pair, tiny_config
from workload import configs

pytestmark = pytest.mark.gpu

SIZES = [5, 300001, 77, 70001]


def _one_ulp(a, i):
    a[i] = np.nextafter(a[i], np.float32(np.inf))


def _planted(ora, what):
    blk = ora.blocks[(0, 1)]                      # the 300,001-element block: 37 chunks
    if what == "params, interior chunk":
        _one_ulp(blk.p, 123457)
    elif what == "params, last element":
        _one_ulp(blk.p, blk.nelem - 1)
    elif what == "state0":
        _one_ulp(blk.s0, 200000)
    elif what == "state1":
        _one_ulp(blk.s1, 8192)
    elif what == "step":
        blk.step += 1
    elif what == "norm":
        blk.sqnorm *= 1.0 + 5e-5
    elif what == "context":
        blk.ctx = 1 - blk.ctx
    else:
        raise AssertionError(what)


WHAT = ["params, interior chunk", "params, last element", "state0", "state1", "step", "norm", "context"]


@pytest.mark.parametrize("what", WHAT)
def test_pair_compare_notices(what):
    cfg = tiny_config(SIZES, 3, opt=configs.ADAM)
    cfg.num_contexts = 2
    pair = Pair(cfg)
    try:
        pair.push_iteration(0)
        pair.aggregate(configs.rounds_all(cfg)[0])
        pair.compare()                            # clean
        _planted(pair.ora, what)
        with pytest.raises(AssertionError):
            pair.compare()
    finally:
        pair.close()


@pytest.mark.parametrize("what", WHAT)
def test_full_pair_compare_notices(what):
    cfg = tiny_config(SIZES, 3, opt=configs.ADAM)
    cfg.num_contexts = 2
    pair = FullPair(cfg)
    try:
        pair.iteration(0, configs.rounds_all(cfg))
        assert pair.compare(1) == cfg.num_params  # clean
        _planted(pair.ora, what)
        with pytest.raises(AssertionError):
            pair.compare(1)
    finally:
        pair.close()


def test_padding_check_notices_a_write_past_the_last_element():
    """The bytes between a block's last element and the end of its 256-byte
    section must stay zero; the check reads them from the device.  Here the
    test itself writes one float there (through a view of the arena, as a
    kernel overrun would) and the check has to see it."""
    cfg = tiny_config([5, 77], 2)
    pair = Pair(cfg)
    try:
        pair.push_iteration(0)
        pair.aggregate(configs.rounds_all(cfg)[0])
        pair.compare()
        pair.check_padding(0, 0, 5, 2, "clean")
        base = pair.svc.pull(0, 0)
        pair.svc.view(base + 4 * 5, 1).fill_(1.0)                 # element 5 of a 5-element block: padding
        torch.cuda.synchronize()
        with pytest.raises(AssertionError):
            pair.check_padding(0, 0, 5, 2, "planted")
    finally:
        pair.close()
