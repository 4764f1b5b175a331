"""Shapes, block cutting, arrival schedules and seeded generators."""
import numpy as np
import torch

from workload import configs, generate, shapes


def test_model_parameter_and_tensor_counts():
    want = {"alexnet": (16, 61_100_840), "vgg16": (32, 138_357_544), "resnet50": (161, 25_557_032),
            "awd_lm": (14, 24_240_478), "bert_base": (199, 109_482_240), "bert_large": (393, 335_143_938)}
    for name, (nt, npar) in want.items():
        t = shapes.MODELS[name]()
        assert len(t) == nt and shapes.num_params(t) == npar, name


def test_block_counts_and_round_bytes():
    c = {n: f() for n, f in configs.CONFIGS.items()}
    assert [len(j.blocks) for j in c["C1"].jobs] == [16]
    assert len(c["C2"].jobs[0].blocks) == 169
    assert len(c["C3"].jobs[0].blocks) == 147
    assert len(c["C5"].jobs[0].blocks) == 566
    assert c["C4"].num_params == 661_141_770 and len(c["C4"].jobs) == 12
    assert [j.num_workers for j in c["C4"].jobs] == [2, 4, 8, 16] * 3
    assert c["C1"].bytes_per_round() == 33_554_432            # (4+4)*4 * 2^20
    assert c["C2"].bytes_per_round() == (8 + 4) * 4 * 25_557_032
    assert c["C3"].bytes_per_round() == (16 + 4) * 4 * 138_357_544
    assert c["C5"].bytes_per_round() == (2 * 32 + 24) * 335_143_938
    assert abs(c["C4"].bytes_per_round() - 31.03e9) < 0.01e9


def test_blocks_tile_each_job_exactly():
    for f in configs.CONFIGS.values():
        for job in f().jobs:
            off = 0
            for b in job.blocks:
                assert b.job_offset == off and 0 < b.nelem
                off += b.nelem
            assert off == job.num_params
    c3 = configs.c3().jobs[0]
    assert all(b.nelem <= shapes.BLOCK_ELEMS or c3.tensors[b.tensor].name.startswith("conv") for b in c3.blocks)


def test_every_task_arrives_exactly_once_per_iteration():
    for name in ("C2", "C4", "C5"):
        cfg = configs.CONFIGS[name]()
        every = sorted((j, b.block) for j, job in enumerate(cfg.jobs) for b in job.blocks)
        for it in range(2):
            rounds = configs.rounds_for(cfg, it)
            assert sorted(t for r in rounds for t in r) == every
    c2 = configs.c2()
    first = configs.rounds_for(c2, 0)[0]
    last_layer = max(b.layer for b in c2.jobs[0].blocks)
    assert all(c2.jobs[0].blocks[b].layer == last_layer for _, b in first)   # fc first


def test_poisson_rounds_are_seeded_and_bursty():
    cfg = configs.c4()
    a, b = configs.rounds_for(cfg, 0), configs.rounds_for(cfg, 0)
    assert a == b and a != configs.rounds_for(cfg, 1)
    sizes = [len(r) for r in a]
    assert max(sizes) > 2 * min(sizes)
    # within a job, layers become ready last-to-first
    t = configs.arrival_times_poisson(cfg, 0)
    for j, job in enumerate(cfg.jobs):
        layers = [job.blocks[b].layer for _, jj, b in t if jj == j]
        assert layers == sorted(layers, reverse=True)


def test_generators_are_deterministic_and_shaped():
    cfg = configs.c1()
    g0, g0b, g1 = generate.grad_slab(cfg, 0, 0), generate.grad_slab(cfg, 0, 0), generate.grad_slab(cfg, 0, 1)
    assert torch.equal(g0, g0b) and not torch.equal(g0, g1)
    assert g0.shape == (4, 1 << 20) and abs(g0.std().item() - 1e-2) < 1e-4
    p = generate.init_params(cfg, 0)
    assert abs(p.std().item() - 0.05) < 1e-3
    # every worker draws its own gradients (identical shards would hide a wrong worker order or a
    # dropped worker from every parity test), and they are uncorrelated
    for a in range(4):
        for b in range(a + 1, 4):
            assert not torch.equal(g0[a], g0[b])
            assert abs(float((g0[a] * g0[b]).mean()) / 1e-4) < 0.01
    assert abs(g0.mean().item()) < 1e-4 and (g0 != 0).float().mean() > 0.999


def test_row_sparse_embedding_and_bf16_rounding():
    cfg = configs.c4()
    cfg.jobs = [cfg.jobs[6]]                  # one AWD-LM-shaped job
    job = cfg.jobs[0]
    g = generate.grad_slab(cfg, 0, 0)
    emb = g[:, :33278 * 400].view(job.num_workers, 33278, 400)
    frac = (emb.abs().sum(-1) > 0).float().mean(-1)
    assert torch.all((frac > 0.04) & (frac < 0.06))
    assert (g[:, 33278 * 400:] != 0).float().mean() > 0.99
    c5 = configs.c5()
    c5.jobs[0].tensors = c5.jobs[0].tensors[3:5]
    c5.jobs[0].blocks = shapes.cut_blocks(c5.jobs[0].tensors)
    c5.jobs[0].num_workers = 3
    r, full = generate.grad_slab(c5, 0, 0, keep_fp32=True)
    assert r.dtype == torch.bfloat16 and torch.equal(r, full.to(torch.bfloat16))
    assert torch.max((r.float() - full).abs() / full.abs().clamp_min(1e-30)) <= 2.0 ** -8


def test_migration_plan_is_a_seeded_quarter():
    cfg = configs.c5()
    plan = configs.migration_plan(cfg)
    assert plan == configs.migration_plan(cfg)
    assert len(plan) == round(0.25 * 566) and len(set(plan)) == len(plan)


def test_sample_positions_cover_block_edges():
    cfg = configs.c2()
    pos = generate.sample_positions(cfg, 0, 8).numpy()
    for b in cfg.jobs[0].blocks:
        assert b.job_offset in pos and b.job_offset + b.nelem - 1 in pos
    assert np.all(np.diff(pos) >= 0) and pos.max() < cfg.jobs[0].num_params
