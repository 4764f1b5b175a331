"""Per-task device-time profile (the e_t the paper's assignment scheme takes
as input): present only when asked for, consistent with the launch's wall
time, larger for larger tasks, and without effect on the results."""
import numpy as np
import pytest
import torch

from helpers import Pair, tiny_config
from paper_2204_03211_b200 import binding as B
from workload import configs

pytestmark = pytest.mark.gpu


def test_profile_off_by_default_and_consistent_when_on():
    sizes = [1 << 20, 1 << 18, 4096, 3 << 20]
    cfg = tiny_config(sizes, 8)
    pair = Pair(cfg)
    svc = pair.svc
    try:
        every = configs.rounds_all(cfg)[0]
        pair.push_iteration(0)
        pair.aggregate(every)
        torch.cuda.synchronize()
        assert svc.block_profile(0, 0) == (0.0, 0.0) and svc.job_profile(0) == (0.0, 0.0, 0)

        svc.set_option(B.PS_OPT_PROFILE, 1)
        pair.push_iteration(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        pair.aggregate(every)
        e1.record()
        torch.cuda.synchronize()
        wall_us = e0.elapsed_time(e1) * 1e3
        prof = [svc.block_profile(0, b) for b in range(4)]
        busy = [p[0] for p in prof]
        span = [p[1] for p in prof]
        assert all(x > 0 for x in busy) and all(x > 0 for x in span)
        assert busy[3] > busy[0] > busy[1] > busy[2]            # ordered like the sizes
        assert max(span) <= wall_us * 1.05 + 5.0                # no task outlasts the launch
        grid = svc.launch_info()["grid"]
        jb, js, jn = svc.job_profile(0)
        assert jn == 4 and abs(jb - sum(busy)) < 1e-6
        assert jb <= grid * (wall_us * 1.05 + 5.0)              # CTA-time cannot exceed CTAs x wall time
        assert js <= wall_us * 1.05 + 5.0 and js >= max(span) - 1e-6
        pair.compare()                                          # results are untouched by profiling

        svc.set_option(B.PS_OPT_PROFILE, 0)
        pair.push_iteration(2)
        pair.aggregate(every)
        torch.cuda.synchronize()
        assert svc.block_profile(0, 0) == (0.0, 0.0)
        pair.compare()
    finally:
        pair.close()
