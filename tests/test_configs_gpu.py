"""The five benchmark configurations at full size, CUDA path vs CPU oracle.

C1 and C2 are compared in full (every element of every block); C3, C4 and C5
are too large for the oracle to follow whole within seconds, so every block is
checked at a seeded sample of positions (edges, chunk boundaries, interior)
plus a few whole blocks per job — the update is element-wise, so the oracle's
values at those positions are exact.  Launch configuration = the library's
defaults, which is what bench.py times.
"""
import numpy as np
import pytest
import torch

from helpers import Pair, SampledPair
from workload import configs

pytestmark = pytest.mark.gpu


def test_c2_resnet50_shaped_reverse_layer_arrival_50_iterations():
    cfg = configs.c2()
    pair = SampledPair(cfg, per_block=256, full_per_job=4)
    try:
        rounds = configs.rounds_for(cfg, 0)          # fc first, stem last: 54 launches per iteration
        assert len(rounds) == 54
        for it in range(cfg.iterations):
            pair.iteration(it, rounds)
            if it in (0, cfg.iterations - 1):
                pair.compare(it + 1)
    finally:
        pair.close()


def test_c2_all_blocks_in_full_three_iterations_all_at_once():
    cfg = configs.c2()
    pair = Pair(cfg)
    try:
        every = configs.rounds_all(cfg)[0]
        for it in range(3):
            pair.push_iteration(it)
            pair.aggregate(every)
        pair.compare()
    finally:
        pair.close()


def test_c3_vgg16_shaped_20_iterations():
    cfg = configs.c3()
    pair = SampledPair(cfg, per_block=256, full_per_job=4)
    try:
        rounds = configs.rounds_all(cfg)
        for it in range(cfg.iterations):
            pair.iteration(it, rounds)
            if it in (0, cfg.iterations - 1):
                pair.compare(it + 1)
    finally:
        pair.close()


@pytest.mark.parametrize("overlap", [0, 1], ids=["in-stream", "overlapped"])
def test_c4_twelve_packed_jobs_bursty_arrival(overlap):
    from paper_2204_03211_b200 import binding as B
    cfg = configs.c4()
    pair = SampledPair(cfg, per_block=128, full_per_job=4)
    try:
        pair.svc.set_option(B.PS_OPT_OVERLAP, overlap)      # the launch configuration bench.py times is "overlapped"
        stream = torch.cuda.Stream()
        for it in range(cfg.iterations):
            rounds = configs.rounds_for(cfg, it, 16)
            assert all(len({j for j, _ in r}) >= 1 for r in rounds)
            pair.iteration(it, rounds, stream)
            pair.svc.join(stream)
            stream.synchronize()
        pair.compare(cfg.iterations)
        # one more iteration with everything ready at once: a single packed launch
        before = pair.svc.launch_info()["launches"]
        pair.iteration(cfg.iterations, configs.rounds_all(cfg), stream)
        pair.svc.join(stream)
        stream.synchronize()
        assert pair.svc.launch_info()["launches"] == before + 1
        pair.compare(cfg.iterations + 1)
    finally:
        pair.close()


def test_c5_bert_large_shaped_adam_bf16_with_migration():
    cfg = configs.c5()
    pair = SampledPair(cfg, per_block=128, full_per_job=4)
    try:
        rounds = configs.rounds_all(cfg)
        plan = configs.migration_plan(cfg)
        side = torch.cuda.Stream()
        for it in range(cfg.iterations):
            pair.iteration(it, rounds)
            if it == 0:
                pair.compare(1)
            if it + 1 == cfg.migrate_after:
                # a quarter of the blocks changes context between two iterations, on another stream
                pair.migrate(plan, side)
        pair.compare(cfg.iterations)
        used = [pair.svc.arena_info(c)[0] for c in range(cfg.num_contexts)]
        assert sum(used) == sum(3 * ((4 * b.nelem + 255) // 256 * 256) for b in cfg.jobs[0].blocks)
    finally:
        pair.close()
