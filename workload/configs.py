"""The five benchmark configurations as plain data, and their arrival schedules.

Holds shapes, hyper-parameters, seeds and arrival ORDER only; none of the
aggregation arithmetic.  Both the CPU oracle's tests and the CUDA library's
tests/bench build their jobs from these records.

Readings where the configuration text leaves a choice open:
  * N(0, x): x is the standard deviation.
  * C2 has no lr -> 0.1.  C3 has neither lr nor wd -> lr 0.1, wd 0.
  * C4: every job SGD lr 0.1 mom 0.9 wd 1e-4, fp32 gradients; job k of the
    order A,A,A,R,R,R,L,L,L,B,B,B gets W = (2,4,8,16)[k mod 4].
  * C5: Adam wd 0; two contexts, blocks split evenly; after iteration 5 a
    seeded quarter of the blocks moves to the other context.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

from . import shapes

SGD, ADAM = 0, 1
F32, BF16 = 0, 1


@dataclass
class JobSpec:
    name: str
    model: str
    tensors: list
    blocks: list
    num_workers: int
    opt: int = SGD
    grad_dtype: int = F32
    lr: float = 0.1
    momentum: float = 0.9
    weight_decay: float = 1e-4
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    grad_scale: float = 1.0
    grad_std: float = 1e-3
    param_std: float = 0.05
    sparse_row_fraction: float = 0.05   # for tensors flagged row_sparse

    @property
    def num_params(self) -> int:
        return sum(b.nelem for b in self.blocks)

    def hparams(self) -> dict:
        return dict(opt=self.opt, grad_dtype=self.grad_dtype, num_workers=self.num_workers,
                    lr=self.lr, momentum=self.momentum, weight_decay=self.weight_decay,
                    beta1=self.beta1, beta2=self.beta2, eps=self.eps, grad_scale=self.grad_scale)

    def bytes_per_elem(self) -> int:
        """Algorithmic HBM bytes per element per aggregate: W gradient reads,
        parameter read+write, each state tensor read+write."""
        g = 2 if self.grad_dtype == BF16 else 4
        nstate = 2 if self.opt == ADAM else 1
        return self.num_workers * g + 8 * (1 + nstate)


@dataclass
class Config:
    name: str
    seed: int
    iterations: int
    jobs: list
    num_contexts: int = 1
    arrival: str = "all"            # "all" | "reverse_layer" | "poisson"
    migrate_after: int = -1         # iteration after which blocks migrate (C5)
    migrate_fraction: float = 0.0
    notes: dict = field(default_factory=dict)

    @property
    def num_params(self) -> int:
        return sum(j.num_params for j in self.jobs)

    def bytes_per_round(self) -> int:
        return sum(j.bytes_per_elem() * j.num_params for j in self.jobs)


def _job(name, model, W, **kw) -> JobSpec:
    tensors = shapes.MODELS[model]()
    keep = kw.pop("keep_whole", lambda t: False)
    return JobSpec(name, model, tensors, shapes.cut_blocks(tensors, keep_whole=keep), W, **kw)


def c1() -> Config:
    tensors = [shapes.Tensor("block%d" % i, (65536,), i) for i in range(16)]
    job = JobSpec("c1", "flat16", tensors, shapes.cut_blocks(tensors), 4,
                  lr=0.1, momentum=0.9, weight_decay=1e-4, grad_std=1e-2)
    return Config("C1", 0, 10, [job])


def c2() -> Config:
    return Config("C2", 2, 50, [_job("resnet50", "resnet50", 8, lr=0.1, momentum=0.9, weight_decay=1e-4)],
                  arrival="reverse_layer")


def c3() -> Config:
    # conv tensors stay single blocks; the fully connected tensors are cut.
    job = _job("vgg16", "vgg16", 16, lr=0.1, momentum=0.9, weight_decay=0.0,
               keep_whole=lambda t: t.name.startswith("conv"))
    return Config("C3", 3, 20, [job])


C4_MODELS = ["alexnet"] * 3 + ["resnet50"] * 3 + ["awd_lm"] * 3 + ["bert_base"] * 3
C4_WORKERS = (2, 4, 8, 16)


def c4() -> Config:
    jobs = [_job("%s#%d" % (m, k), m, C4_WORKERS[k % 4], lr=0.1, momentum=0.9, weight_decay=1e-4)
            for k, m in enumerate(C4_MODELS)]
    return Config("C4", 4, 3, jobs, arrival="poisson")


def c5() -> Config:
    job = _job("bert_large", "bert_large", 32, opt=ADAM, grad_dtype=BF16, lr=1e-4, weight_decay=0.0,
               momentum=0.0)
    return Config("C5", 5, 10, [job], num_contexts=2, migrate_after=5, migrate_fraction=0.25)


CONFIGS = {"C1": c1, "C2": c2, "C3": c3, "C4": c4, "C5": c5}


# --------------------------------------------------------------------------
# Arrival schedules: which (job, block) tasks are ready in which round.
# --------------------------------------------------------------------------

def rounds_all(cfg: Config) -> list:
    """One round holding every task of every job."""
    return [[(j, b.block) for j, job in enumerate(cfg.jobs) for b in job.blocks]]


def rounds_reverse_layer(cfg: Config) -> list:
    """Backward finishes the last layer first: one round per layer, last
    layer's blocks first (within a layer, blocks in reverse id order)."""
    rounds = []
    for j, job in enumerate(cfg.jobs):
        layers = sorted({b.layer for b in job.blocks}, reverse=True)
        for l in layers:
            rounds.append([(j, b.block) for b in reversed(job.blocks) if b.layer == l])
    return rounds


def arrival_times_poisson(cfg: Config, iteration: int, window: float = 1.0) -> list:
    """Per job: the backward pass starts at a seeded offset inside the window
    and emits its layers last-to-first with exponential gaps (a Poisson
    process over layers), compressed to fit the job's own backward duration.
    Returns [(time, job, block)], times in [0, window)."""
    out = []
    for j, job in enumerate(cfg.jobs):
        rng = np.random.default_rng([cfg.seed, 7919, j, iteration])
        duration = window * rng.uniform(0.35, 0.9)
        start = rng.uniform(0.0, window - duration)
        layers = sorted({b.layer for b in job.blocks}, reverse=True)
        gaps = rng.exponential(1.0, size=len(layers))
        t = start + duration * np.cumsum(gaps) / gaps.sum()
        when = {l: float(min(tt, window * (1 - 1e-9))) for l, tt in zip(layers, t)}
        for b in reversed(job.blocks):
            out.append((when[b.layer], j, b.block))
    out.sort(key=lambda x: x[0])
    return out


def rounds_poisson(cfg: Config, iteration: int, ticks: int = 16) -> list:
    """Cuts the virtual clock of one iteration window into `ticks` rounds;
    round r lists the tasks that arrived during tick r.  Every task of every
    job appears in exactly one round; empty rounds are dropped."""
    rounds = [[] for _ in range(ticks)]
    for t, j, b in arrival_times_poisson(cfg, iteration):
        rounds[min(int(t * ticks), ticks - 1)].append((j, b))
    return [r for r in rounds if r]


def rounds_for(cfg: Config, iteration: int, ticks: int = 16) -> list:
    if ticks == 1:          # one round: everything is ready at once, whatever the arrival pattern
        return rounds_all(cfg)
    if cfg.arrival == "reverse_layer":
        return rounds_reverse_layer(cfg)
    if cfg.arrival == "poisson":
        return rounds_poisson(cfg, iteration, ticks)
    return rounds_all(cfg)


def migration_plan(cfg: Config) -> list:
    """[(job, block)] that change context after iteration cfg.migrate_after."""
    if cfg.migrate_after < 0:
        return []
    rng = np.random.default_rng([cfg.seed, 104729])
    plan = []
    for j, job in enumerate(cfg.jobs):
        n = len(job.blocks)
        pick = rng.choice(n, size=max(1, int(round(cfg.migrate_fraction * n))), replace=False)
        plan += [(j, int(b)) for b in sorted(pick)]
    return plan


def initial_context(cfg: Config, job: int, block: int) -> int:
    """Blocks start split evenly over the contexts (round-robin by id)."""
    return block % cfg.num_contexts
