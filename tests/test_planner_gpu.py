"""Profile -> plan -> migrate, end to end on the device: measured per-block
device times (e_t) feed the planner, its Aggregator choices become contexts,
blocks are migrated there, and the numerical results still equal the oracle's."""
import pytest
import torch

from helpers import Pair, tiny_config
from paper_2204_03211_b200 import binding as B
from workload import configs

pytestmark = pytest.mark.gpu


def test_measured_task_times_drive_placement_and_results_are_unchanged():
    sizes = [1 << 19, 1 << 18, 3 << 18, 1 << 17, 1 << 19, 5000, 1 << 18, 1 << 16]
    cfg = tiny_config(sizes, 4)
    cfg.num_contexts = 8
    pair = Pair(cfg)
    svc = pair.svc
    try:
        every = configs.rounds_all(cfg)[0]
        svc.set_option(B.PS_OPT_PROFILE, 1)
        pair.push_iteration(0)
        pair.aggregate(every)
        e = [svc.block_profile(0, b)[0] for b in range(len(sizes))]
        assert all(x > 0 for x in e)
        # an iteration period that one Aggregator cannot cover: the plan must spread the blocks
        D = sum(e) / 2.5
        plan = B.Planner(0.1)
        j = plan.add_job(D)
        where = [plan.assign(j, x)[1] for x in e]
        alloc, alive = plan.num_aggregators()
        assert 3 <= alive <= 8 and alloc == alive
        for n in range(alloc):
            info = plan.aggregator_info(n)
            assert info["load"] <= info["cycle"] + 1e-9 and info["cycle"] == D
        side = torch.cuda.Stream()
        for b, n in enumerate(where):
            pair.migrate(0, b, n, side)
        for it in (1, 2):
            pair.push_iteration(it)
            pair.aggregate(every)
        pair.compare()              # also checks every block's context against the oracle's
        assert [svc.block_state(0, b)[2] for b in range(len(sizes))] == where
    finally:
        pair.close()
