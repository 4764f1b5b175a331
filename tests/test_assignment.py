"""Pins of the assignment oracle (Pseudocode 1 of the paper) and parity of the
library's planner against it.  CPU only."""
import os

import numpy as np
import pytest

from oracle import assignment as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "cyclic_execution_toy.txt")


def _golden():
    out = {}
    for line in open(GOLDEN):
        line = line.split("#")[0].split()
        if len(line) == 2:
            out[line[0]] = float(line[1])
    return out


# ------------------------------------------------------------------ the paper's printed numbers

def test_toy_case_a_cycles_and_repetitions():
    g = _golden()
    o = O.AssignmentOracle(g["loss_limit"])
    j1, j2 = o.add_job(g["A.D1"]), o.add_job(g["A.D2"])
    _, n1 = o.assign(j1, g["A.e1"])
    assert o.cycle(n1) == g["A.cycle_J1_alone"]
    alone = O.AssignmentOracle(g["loss_limit"])
    _, m = alone.assign(alone.add_job(g["A.D2"]), g["A.e2"])
    assert alone.cycle(m) == g["A.cycle_J2_alone"]
    _, n2 = o.assign(j2, g["A.e2"])
    assert n2 == n1                                   # packed onto the same Aggregator
    assert o.cycle(n1) == g["A.cycle_packed"]
    assert O.floor_ratio(o.cycle(n1), o.current_duration(j1)) == g["A.runs_of_J1_per_cycle"]
    assert o.current_duration(j1) == g["A.D1"] and o.current_duration(j2) == g["A.D2"]   # nobody slowed down
    assert o.load(n1) == 2 * g["A.e1"] + g["A.e2"]    # W_n of Appendix C
    assert o.num_alive() == 1


def test_toy_case_b_seventeen_percent_loss_forces_a_new_aggregator():
    g = _golden()
    assert O.stretched_duration(g["B.D"], g["B.cycle_after"]) == g["B.duration_after"]
    assert round(100 * O.loss(g["B.D"], g["B.duration_after"])) == g["B.loss_percent_rounded"]
    o = O.AssignmentOracle(g["loss_limit"])
    a, b = o.add_job(g["B.D"]), o.add_job(g["A.D2"])
    _, n0 = o.assign(a, g["B.e"])
    assert o.estimate(n0, b, g["A.e2"]) is None       # 17 % >= LossLimit: not a destination
    _, n1 = o.assign(b, g["A.e2"])
    assert n1 != n0 and o.num_alive() == 2
    assert o.current_duration(a) == g["B.D"]          # the existing job keeps its speed
    # with a laxer limit the same request is packed and the job is stretched to 6
    lax = O.AssignmentOracle(0.2)
    a, b = lax.add_job(g["B.D"]), lax.add_job(g["A.D2"])
    _, n0 = lax.assign(a, g["B.e"])
    _, n1 = lax.assign(b, g["A.e2"])
    assert n1 == n0 and lax.current_duration(a) == g["B.duration_after"]
    assert lax.cycle(n0) == g["B.cycle_after"]


# ------------------------------------------------------------------ properties of the scheme

def test_free_slot_estimate_matches_appendix_c_load():
    o = O.AssignmentOracle()
    j1, j2 = o.add_job(6), o.add_job(12)
    _, n = o.assign(j1, 2)
    F, need = o.estimate(n, j2, 3)
    assert (F, need) == (12 - 2 * 2, 3)
    o.assign(j2, 3)
    F, need = o.estimate(n, j1, 1.0)
    assert F == 12 - o.load(n) == 5 and need == 2 * 1.0   # a J1 task runs twice per cycle


def test_overload_opens_a_new_aggregator_and_best_fit_picks_the_tightest():
    o = O.AssignmentOracle()
    j = o.add_job(10)
    assert [o.assign(j, 6)[1], o.assign(j, 6)[1]] == [0, 1]       # 6 + 6 > 10
    assert o.assign(j, 3)[1] == 0                                  # both have 4 free: lowest index
    assert o.assign(j, 1)[1] == 0                                  # free: n0 = 1, n1 = 4 -> tightest that fits
    assert o.assign(j, 2)[1] == 1                                  # n0 is full
    assert o.assign(j, 4)[1] == 2                                  # nobody fits
    for n in range(3):
        assert o.load(n) <= o.cycle(n)                             # constraint W_n <= C_n


def test_random_sequences_respect_the_constraints():
    rng = np.random.default_rng(0)
    o = O.AssignmentOracle()
    jobs = [o.add_job(float(rng.choice([5, 6, 10, 12, 20, 24, 25, 60]))) for _ in range(12)]
    for _ in range(300):
        k = int(rng.integers(len(jobs)))
        o.assign(k, float(rng.uniform(0.05, 0.2) * o.D[k]))
    for n, a in enumerate(o.N):
        assert o.load(n) <= o.cycle(n) + 1e-9
    for k in jobs:
        assert O.loss(o.D[k], o.current_duration(k)) < o.loss_limit
    assert len(o.where) == 300


def test_job_exit_releases_and_recycles_aggregators():
    o = O.AssignmentOracle()
    a, b = o.add_job(10), o.add_job(10)
    for _ in range(3):
        o.assign(a, 4)          # a: 4+4 on n0, 4 on n1
    o.assign(b, 5)              # n1: 4 + 5
    o.assign(b, 9)              # n2
    assert o.num_alive() == 3
    released = o.remove_job(b)  # n2 becomes empty; then n1 (load 4) cannot move onto n0 (load 8)
    assert released == 1 and o.num_alive() == 2
    c = o.add_job(10)
    o.assign(c, 1)
    released = o.remove_job(c)
    assert released == 0
    # after a leaves partly... remove a's heavy use: everything of a goes
    assert o.remove_job(a) == 2 and o.num_alive() == 0


def test_recycling_moves_a_light_aggregator_onto_others():
    o = O.AssignmentOracle()
    a, b = o.add_job(10), o.add_job(10)
    o.assign(a, 6)              # n0
    o.assign(b, 6)              # n1 (6 + 6 > 10)
    t, n = o.assign(a, 2)       # n0: 8
    o.assign(b, 3)              # n1: 9
    _, n2 = o.assign(a, 2)      # n0 is the tightest that fits: 10
    assert n2 == 0
    _, n3 = o.assign(b, 2)      # nothing fits -> n2
    assert n3 == 2
    c = o.add_job(10)
    o.assign(c, 1)              # n1 (1 free) is the tightest
    assert o.where[max(o.where)] == 1
    # job b leaves: n1 keeps c's task (1), n2 becomes empty -> released; then n1's
    # single light task cannot go to n0 (full) -> stays
    assert o.remove_job(b) == 1 and o.num_alive() == 2
    # job a leaves: n0 empty -> released; one Aggregator left, nothing to recycle
    assert o.remove_job(a) == 1 and o.num_alive() == 1


def test_outlier_rule():
    # cycle 12, 7 units gone, 3 units of scheduled work still to run: 2 units are spare
    assert O.outlier_fits(12, 7, 3, 2)
    assert not O.outlier_fits(12, 7, 3, 2.5)          # postponed to the next cycle


def test_floor_guard():
    assert O.floor_ratio(12, 6) == 2 and O.floor_ratio(0.3, 0.1) == 3 and O.floor_ratio(11.999, 6) == 1
    assert O.stretched_duration(7, 5) == 7            # a cycle shorter than the period never speeds a job up
