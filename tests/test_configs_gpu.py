"""The five benchmark configurations at full size, CUDA path vs CPU oracle,
every element of every block.

The oracle follows all iterations in full: each iteration's gradients are
generated on the GPU and handed to it as host copies, one job's slab at a time;
after the first and the last iteration (C5: also after the first one that
follows the migration) every element of parameters and optimizer state is
compared bit for bit, and every block's step, context and gradient norm.
Launch configuration = the one bench.py times: overlapped launches, rounds
given with their inputs complete, packing over time.  C2's 50-iteration
layer-by-layer replay additionally runs with the sampled checker, as a second,
independent path through the comparison code.
"""
import numpy as np
import pytest
import torch

from helpers import FullPair, Pair, SampledPair
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


def test_c2_layer_by_layer_in_full_every_element():
    cfg = configs.c2()
    pair = FullPair(cfg)
    try:
        rounds = configs.rounds_for(cfg, 0)
        for it in range(cfg.iterations):
            pair.iteration(it, rounds)
            if it in (0, cfg.iterations - 1):
                assert pair.compare(it + 1) == cfg.num_params
    finally:
        pair.close()


def test_c3_vgg16_shaped_20_iterations_every_element():
    cfg = configs.c3()
    pair = FullPair(cfg)
    try:
        rounds = configs.rounds_all(cfg)
        for it in range(cfg.iterations):
            pair.iteration(it, rounds)
            if it in (0, cfg.iterations - 1):
                assert pair.compare(it + 1) == cfg.num_params
    finally:
        pair.close()


@pytest.mark.parametrize("name", ["C3", "C5"])
def test_ring_kernel_on_full_size_shapes_every_element(name):
    """The bulk-copy ring kernel (PS_OPT_KERNEL = 2) on the VGG-16-shaped job (fp32, SGD, W = 16)
    and the BERT-large-shaped one (bf16, Adam, W = 32, two contexts): three iterations, every
    element and every block's norm compared after the first and the last — full-size launches
    are where a CTA closes hundreds of chunks and its publisher warp draws tickets in batches."""
    cfg = configs.CONFIGS[name]()
    pair = FullPair(cfg, kernel=2)
    try:
        rounds = configs.rounds_all(cfg)
        for it in range(3):
            pair.iteration(it, rounds)
            if it in (0, 2):
                assert pair.compare(it + 1) == cfg.num_params
        assert pair.svc.launch_info()["kernel"] == "bulk"
    finally:
        pair.close()


@pytest.mark.parametrize("overlap", [0, 1], ids=["in-stream", "overlapped"])
def test_c4_twelve_packed_jobs_bursty_arrival_every_element(overlap):
    cfg = configs.c4()
    pair = FullPair(cfg, overlap=overlap)       # the launch configuration bench.py times is "overlapped"
    try:
        for it in range(cfg.iterations):
            rounds = configs.rounds_for(cfg, it, 16)
            pair.iteration(it, rounds)
            if it in (0, cfg.iterations - 1):
                assert pair.compare(it + 1) == cfg.num_params
        # one more iteration with everything ready at once: a single packed round
        before = pair.svc.launch_info()["launches"]
        pair.iteration(cfg.iterations, configs.rounds_all(cfg))
        # in the caller's stream: one launch; overlapped: up to four, whose tails and heads overlap
        assert before + 1 <= pair.svc.launch_info()["launches"] <= before + (4 if overlap else 1)
        pair.compare(cfg.iterations + 1)
    finally:
        pair.close()


def test_c5_bert_large_shaped_adam_bf16_with_migration_every_element():
    cfg = configs.c5()
    pair = FullPair(cfg)
    try:
        rounds = configs.rounds_all(cfg)
        plan = configs.migration_plan(cfg)
        side = torch.cuda.Stream()
        for it in range(cfg.iterations):
            pair.iteration(it, rounds)
            if it in (0, cfg.migrate_after, cfg.iterations - 1):     # first, first after the migration, last
                assert pair.compare(it + 1) == cfg.num_params
            if it + 1 == cfg.migrate_after:
                # a quarter of the blocks changes context between two iterations, on another stream
                pair.migrate(plan, side)
        used = [pair.svc.arena_info(c)[0] for c in range(cfg.num_contexts)]
        assert sum(used) == sum(3 * ((4 * b.nelem + 255) // 256 * 256) for b in cfg.jobs[0].blocks)
    finally:
        pair.close()
