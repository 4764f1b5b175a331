"""CPU oracle of the model-aggregation ASSIGNMENT scheme (TEST INFRASTRUCTURE ONLY).

Follows the paper's Pseudocode 1 ("Model Aggregation Assignment Scheme",
Section 3.3.1) step by step in the paper's notation, with the formulas of
Appendix C ("Problem Definition of Model Aggregation Assignment") for the
quantities both share, the recycling rule of Section 3.3.2 ("Aggregator
Scaling") for job exit, and the outlier rule of Section 3.3.1 ("Handling
Outliers in Cyclic Execution").  Plain Python floats (binary64); no code is
shared with the library's planner.

Notation (Table 1):  C_n execution cycle of Aggregator n;  D_j profiled
iteration duration of job j;  d_j current iteration duration of job j;
e_t execution time of task t;  F_n^est estimated free slots on n;  J_n jobs with
tasks on n;  T_j^n tasks of job j on n.

Readings where the printed pseudocode is garbled or silent:
  * C_n^new in the free-slot line is C_n^est (no other quantity is defined).
  * "N <- N ∩ s" / "T <- T ∩ t" are unions (adding an element).
  * The loss test is applied to every job j of the inner loop, and the job k of
    the new task is examined too (k's own tasks would be stretched by a longer
    cycle; the paper's principle is that no job loses performance by sharing).
  * A task of job k placed on n runs floor(C_n^est / d_k) times per cycle, so it
    needs that many times e_t free slots — the multiplicity the load W_n carries
    in Appendix C; it equals the printed "F >= e_t" when the task runs once.
  * Best fit = among the Aggregators with enough free slots, the one with the
    fewest; ties go to the lowest index.
  * floor(a / b) is taken with a relative guard of 1e-9 so that ratios that are
    integers in exact arithmetic (12 / 6, 0.3 / 0.1) do not fall below them.

Pinned (tests/test_assignment.py) by the numbers the paper prints for its toy
example: J1 (D = 6, e = 2) and J2 (D = 12, e = 3) packed give a cycle of 12 with
J1 run twice; a task with e = 1, D = 5 joined by J2's task gets d = 6 and a loss
of 17 %.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

LOSS_LIMIT = 0.1   # LossLimit, the paper's default


def floor_ratio(a: float, b: float) -> int:
    return int(math.floor(a / b * (1.0 + 1e-9) + 1e-12))


def stretched_duration(D_j: float, C: float) -> float:
    """d_j = max(D_j, C / floor(C / D_j)): a job whose period divides the cycle
    r times gets a slot every C / r."""
    r = floor_ratio(C, D_j)
    return D_j if r < 1 else max(D_j, C / r)


def loss(D_j: float, d_j: float) -> float:
    """L_j = (d_j - D_j) / d_j   (Appendix C)."""
    return (d_j - D_j) / d_j


@dataclass
class Aggregator:
    tasks: dict = field(default_factory=dict)     # job -> {task id: e_t}   (T_j^n)
    alive: bool = True

    def jobs(self):
        return [j for j, ts in self.tasks.items() if ts]


class AssignmentOracle:
    def __init__(self, loss_limit: float = LOSS_LIMIT):
        self.loss_limit = loss_limit
        self.D: list[float] = []                  # D_j
        self.N: list[Aggregator] = []             # allocated Aggregators (dead ones keep their index)
        self.where: dict = {}                     # task id -> Aggregator index
        self.task_job: dict = {}
        self.task_e: dict = {}
        self._next_task = 0

    # ---- quantities of Table 1 / Appendix C
    def cycle(self, n: int) -> float:
        js = self.N[n].jobs()
        return max((self.D[j] for j in js), default=0.0)

    def load(self, n: int) -> float:
        """W_n = sum_j floor(C_n / d_j) * sum_{t in T_j^n} e_t with d_j from this Aggregator's cycle."""
        C = self.cycle(n)
        tot = 0.0
        for j in self.N[n].jobs():
            d = stretched_duration(self.D[j], C)
            tot += floor_ratio(C, d) * sum(self.N[n].tasks[j].values())
        return tot

    def current_duration(self, j: int) -> float:
        """d_j = max over the Aggregators that hold tasks of j."""
        d = self.D[j]
        for n, a in enumerate(self.N):
            if a.alive and a.tasks.get(j):
                d = max(d, stretched_duration(self.D[j], self.cycle(n)))
        return d

    # ---- registration
    def add_job(self, D_j: float) -> int:
        if not D_j > 0:
            raise ValueError("D_j must be positive")
        self.D.append(float(D_j))
        return len(self.D) - 1

    # ---- Pseudocode 1
    def estimate(self, n: int, k: int, e_t: float):
        """The estimate block of the pseudocode for Aggregator n: returns None if
        n is removed from the destinations, else (F_n^est, slots the task needs)."""
        C_est = max(self.cycle(n), self.D[k])
        free = C_est
        for j in sorted(set(self.N[n].jobs()) | {k}):
            d_j = stretched_duration(self.D[j], C_est)
            if loss(self.D[j], d_j) >= self.loss_limit:
                return None
            free -= floor_ratio(C_est, d_j) * sum(self.N[n].tasks.get(j, {}).values())
        need = floor_ratio(C_est, stretched_duration(self.D[k], C_est)) * e_t
        return free, need

    def _place(self, n: int, k: int, e_t: float, task: int | None = None) -> int:
        if task is None:
            task = self._next_task
            self._next_task += 1
        self.N[n].tasks.setdefault(k, {})[task] = e_t
        self.where[task], self.task_job[task], self.task_e[task] = n, k, e_t
        return task

    def choose(self, k: int, e_t: float, allow_new: bool = True, exclude: int = -1):
        best = None
        for n, a in enumerate(self.N):
            if not a.alive or n == exclude:
                continue
            est = self.estimate(n, k, e_t)
            if est is None:
                continue
            F, need = est
            if F >= need - 1e-12 and (best is None or F < best[1]):
                best = (n, F)
        if best is not None:
            return best[0]
        if not allow_new:
            return None
        self.N.append(Aggregator())
        return len(self.N) - 1

    def assign(self, k: int, e_t: float):
        """Returns (task id, Aggregator index)."""
        if not e_t > 0:
            raise ValueError("e_t must be positive")
        n = self.choose(k, e_t)
        return self._place(n, k, e_t), n

    # ---- Section 3.3.2: job exit, recycle lightly loaded Aggregators
    def remove_job(self, k: int) -> int:
        """Removes job k's tasks, releases empty Aggregators, then tries to empty
        the least-loaded ones by re-assigning their tasks elsewhere without new
        allocations.  Returns the number of Aggregators released."""
        released = 0
        for t in [t for t, j in self.task_job.items() if j == k]:
            n = self.where.pop(t)
            del self.N[n].tasks[k][t]
            del self.task_job[t], self.task_e[t]
        for a in self.N:
            if a.alive and not a.jobs():
                a.alive = False
                released += 1
        while True:
            live = [n for n, a in enumerate(self.N) if a.alive]
            if len(live) < 2:
                break
            n = min(live, key=lambda i: (self.load(i), i))
            moved = []
            ok = True
            for j in sorted(self.N[n].jobs()):
                for t, e in sorted(self.N[n].tasks[j].items()):
                    dst = self.choose(j, e, allow_new=False, exclude=n)
                    if dst is None:
                        ok = False
                        break
                    del self.N[n].tasks[j][t]
                    self._place(dst, j, e, task=t)
                    moved.append((t, j, e, dst))
                if not ok:
                    break
            if not ok:
                for t, j, e, dst in reversed(moved):     # revert
                    del self.N[dst].tasks[j][t]
                    self._place(n, j, e, task=t)
                break
            self.N[n].alive = False
            released += 1
        return released

    def num_alive(self) -> int:
        return sum(a.alive for a in self.N)


def outlier_fits(C_n: float, now_in_cycle: float, remaining_scheduled: float, e_late: float) -> bool:
    """A request that missed its slot runs in the current cycle only if enough
    slots remain after reserving those of the requests still scheduled in it;
    otherwise it is postponed to the next cycle."""
    return (C_n - now_in_cycle) - remaining_scheduled >= e_late - 1e-12
