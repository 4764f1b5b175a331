// Host-side planner: which Aggregator (context) should run which aggregation
// task.  Implements the paper's assignment heuristic (Section 3.3.1, Pseudocode 1
// "Model Aggregation Assignment Scheme"), cyclic execution, the recycling of
// lightly loaded Aggregators on job exit (Section 3.3.2) and the rule for late
// requests ("Handling Outliers in Cyclic Execution").  Pure host code; its
// inputs e_t and D_j come from the profiler (ps_block_profile) and the caller.
//
// State per Aggregator n: for every job j with tasks on n the sum S[n][j] of
// their execution times — all the scheme needs, since C_n, d_j, W_n and F_n are
// functions of the D_j and those sums (Appendix C):
//   C_n  = max_{j on n} D_j
//   d_j  = max(D_j, C / floor(C / D_j))
//   W_n  = sum_j floor(C_n / d_j) * S[n][j]
//   loss = (d_j - D_j) / d_j
#include "../../include/ps_b200.h"

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <map>
#include <mutex>
#include <new>
#include <vector>

namespace {

constexpr uint32_t kPlannerMagic = 0x50504c4eu;   // "PPLN"

// floor(a / b) with a relative guard, so that quotients that are whole numbers
// in exact arithmetic are not rounded below themselves.
long long floor_div(double a, double b) { return (long long)std::floor(a / b * (1.0 + 1e-9) + 1e-12); }

double stretched(double D, double C) {
  const long long r = floor_div(C, D);
  return r < 1 ? D : std::max(D, C / (double)r);
}

struct Task {
  int job = -1, agg = -1;
  double e = 0.0;
  bool alive = false;
};

struct Agg {
  bool alive = true;
  std::map<int, double> sum;     // job -> sum of e_t of its tasks here
  std::map<int, int> count;      // job -> number of tasks here
};

}  // namespace

struct ps_planner {
  uint32_t magic = kPlannerMagic;
  double loss_limit = 0.1;
  std::mutex mu;
  std::vector<double> D;
  std::vector<Task> tasks;
  std::vector<Agg> aggs;

  double cycle(int n) const {
    double c = 0.0;
    for (auto& kv : aggs[n].count)
      if (kv.second > 0) c = std::max(c, D[kv.first]);
    return c;
  }
  double load(int n) const {
    const double C = cycle(n);
    double w = 0.0;
    for (auto& kv : aggs[n].count)
      if (kv.second > 0) w += (double)floor_div(C, stretched(D[kv.first], C)) * aggs[n].sum.at(kv.first);
    return w;
  }
  // Estimate block of Pseudocode 1 for one Aggregator.  false = not a destination.
  bool estimate(int n, int k, double e, double* free_out, double* need_out) const {
    const double C = std::max(cycle(n), D[k]);
    double free_slots = C;
    bool k_seen = false;
    for (auto& kv : aggs[n].count) {
      if (kv.second <= 0) continue;
      const int j = kv.first;
      k_seen |= (j == k);
      const double d = stretched(D[j], C);
      if ((d - D[j]) / d >= loss_limit) return false;
      free_slots -= (double)floor_div(C, d) * aggs[n].sum.at(j);
    }
    const double dk = stretched(D[k], C);
    if (!k_seen && (dk - D[k]) / dk >= loss_limit) return false;
    *free_out = free_slots;
    *need_out = (double)floor_div(C, dk) * e;
    return true;
  }
  // Best fit among the live Aggregators (fewest free slots that still suffice,
  // lowest index on ties); -1 if none qualifies.
  int best_fit(int k, double e, int exclude) const {
    int best = -1;
    double best_free = 0.0;
    for (int n = 0; n < (int)aggs.size(); ++n) {
      if (!aggs[n].alive || n == exclude) continue;
      double f, need;
      if (!estimate(n, k, e, &f, &need)) continue;
      if (f >= need - 1e-12 && (best < 0 || f < best_free)) {
        best = n;
        best_free = f;
      }
    }
    return best;
  }
  void put(int t, int n) {
    Task& T = tasks[t];
    T.agg = n;
    aggs[n].sum[T.job] += T.e;
    aggs[n].count[T.job] += 1;
  }
  void take(int t) {
    Task& T = tasks[t];
    Agg& a = aggs[T.agg];
    if (--a.count[T.job] == 0) {
      a.count.erase(T.job);
      a.sum.erase(T.job);
    } else {
      // recompute the sum from the remaining tasks: no drift from repeated subtraction
      double s = 0.0;
      for (const Task& o : tasks)
        if (o.alive && &o != &T && o.agg == T.agg && o.job == T.job) s += o.e;
      a.sum[T.job] = s;
    }
    T.agg = -1;
  }
  bool empty(int n) const { return aggs[n].count.empty(); }
};

namespace {
bool ok(const ps_planner* p) { return p && p->magic == kPlannerMagic; }
}

extern "C" {

int ps_planner_create(ps_planner** out, double loss_limit) {
  if (!out || !(loss_limit > 0.0) || loss_limit > 1.0) return PS_ERR_BAD_ARG;
  ps_planner* p = new (std::nothrow) ps_planner();
  if (!p) return PS_ERR_NOMEM;
  p->loss_limit = loss_limit;
  *out = p;
  return PS_OK;
}

int ps_planner_destroy(ps_planner* p) {
  if (!ok(p)) return PS_ERR_BAD_HANDLE;
  p->magic = 0;
  delete p;
  return PS_OK;
}

int ps_planner_add_job(ps_planner* p, double iter_duration, int* job_out) {
  if (!ok(p)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(p->mu);
  if (!(iter_duration > 0.0) || !job_out) return PS_ERR_BAD_ARG;
  p->D.push_back(iter_duration);
  *job_out = (int)p->D.size() - 1;
  return PS_OK;
}

int ps_planner_assign(ps_planner* p, int job, double exec_time, int* task_out, int* aggregator_out) {
  if (!ok(p)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(p->mu);
  if (job < 0 || job >= (int)p->D.size() || !(exec_time > 0.0)) return PS_ERR_BAD_ARG;
  int n = p->best_fit(job, exec_time, -1);
  if (n < 0) {                       // no destination qualifies: allocate a new Aggregator
    p->aggs.emplace_back();
    n = (int)p->aggs.size() - 1;
  }
  Task t;
  t.job = job; t.e = exec_time; t.alive = true;
  p->tasks.push_back(t);
  const int id = (int)p->tasks.size() - 1;
  p->put(id, n);
  if (task_out) *task_out = id;
  if (aggregator_out) *aggregator_out = n;
  return PS_OK;
}

int ps_planner_remove_job(ps_planner* p, int job, int* released_out) {
  if (!ok(p)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(p->mu);
  if (job < 0 || job >= (int)p->D.size()) return PS_ERR_BAD_ARG;
  int released = 0;
  for (int t = 0; t < (int)p->tasks.size(); ++t)
    if (p->tasks[t].alive && p->tasks[t].job == job) {
      p->take(t);
      p->tasks[t].alive = false;
    }
  for (auto& a : p->aggs)
    if (a.alive && a.count.empty()) { a.alive = false; ++released; }
  // recycle: empty the least-loaded Aggregator onto the others, no new allocation
  while (true) {
    int live = 0, pick = -1;
    double pick_load = 0.0;
    for (int n = 0; n < (int)p->aggs.size(); ++n) {
      if (!p->aggs[n].alive) continue;
      ++live;
      const double w = p->load(n);
      if (pick < 0 || w < pick_load) { pick = n; pick_load = w; }
    }
    if (live < 2) break;
    std::vector<int> here;                      // its tasks, by (job, task id)
    for (int t = 0; t < (int)p->tasks.size(); ++t)
      if (p->tasks[t].alive && p->tasks[t].agg == pick) here.push_back(t);
    std::stable_sort(here.begin(), here.end(), [&](int a, int b) { return p->tasks[a].job < p->tasks[b].job; });
    std::vector<int> moved;
    bool all = true;
    for (int t : here) {
      p->take(t);
      const int dst = p->best_fit(p->tasks[t].job, p->tasks[t].e, pick);
      if (dst < 0) {
        p->put(t, pick);
        all = false;
        break;
      }
      p->put(t, dst);
      moved.push_back(t);
    }
    if (!all) {
      for (auto it = moved.rbegin(); it != moved.rend(); ++it) {
        p->take(*it);
        p->put(*it, pick);
      }
      break;
    }
    p->aggs[pick].alive = false;
    ++released;
  }
  if (released_out) *released_out = released;
  return PS_OK;
}

int ps_planner_task_info(ps_planner* p, int task, int* job_out, int* aggregator_out, double* exec_time_out) {
  if (!ok(p)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(p->mu);
  if (task < 0 || task >= (int)p->tasks.size() || !p->tasks[task].alive) return PS_ERR_BAD_ARG;
  if (job_out) *job_out = p->tasks[task].job;
  if (aggregator_out) *aggregator_out = p->tasks[task].agg;
  if (exec_time_out) *exec_time_out = p->tasks[task].e;
  return PS_OK;
}

int ps_planner_task_runs(ps_planner* p, int task, int* runs_per_cycle_out, double* slot_period_out) {
  if (!ok(p)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(p->mu);
  if (task < 0 || task >= (int)p->tasks.size() || !p->tasks[task].alive) return PS_ERR_BAD_ARG;
  const Task& t = p->tasks[task];
  const double C = p->cycle(t.agg);
  const double d = stretched(p->D[t.job], C);
  if (runs_per_cycle_out) *runs_per_cycle_out = (int)floor_div(C, d);
  if (slot_period_out) *slot_period_out = d;
  return PS_OK;
}

int ps_planner_aggregator_info(ps_planner* p, int aggregator, int* alive_out, double* cycle_out, double* load_out,
                               int* num_tasks_out) {
  if (!ok(p)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(p->mu);
  if (aggregator < 0 || aggregator >= (int)p->aggs.size()) return PS_ERR_BAD_ARG;
  if (alive_out) *alive_out = p->aggs[aggregator].alive ? 1 : 0;
  if (cycle_out) *cycle_out = p->cycle(aggregator);
  if (load_out) *load_out = p->load(aggregator);
  if (num_tasks_out) {
    int c = 0;
    for (auto& kv : p->aggs[aggregator].count) c += kv.second;
    *num_tasks_out = c;
  }
  return PS_OK;
}

int ps_planner_job_info(ps_planner* p, int job, double* profiled_out, double* current_out, double* loss_out) {
  if (!ok(p)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(p->mu);
  if (job < 0 || job >= (int)p->D.size()) return PS_ERR_BAD_ARG;
  double d = p->D[job];
  for (int n = 0; n < (int)p->aggs.size(); ++n) {
    if (!p->aggs[n].alive) continue;
    auto it = p->aggs[n].count.find(job);
    if (it != p->aggs[n].count.end() && it->second > 0) d = std::max(d, stretched(p->D[job], p->cycle(n)));
  }
  if (profiled_out) *profiled_out = p->D[job];
  if (current_out) *current_out = d;
  if (loss_out) *loss_out = (d - p->D[job]) / d;
  return PS_OK;
}

int ps_planner_num_aggregators(ps_planner* p, int* allocated_out, int* alive_out) {
  if (!ok(p)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(p->mu);
  int alive = 0;
  for (auto& a : p->aggs) alive += a.alive ? 1 : 0;
  if (allocated_out) *allocated_out = (int)p->aggs.size();
  if (alive_out) *alive_out = alive;
  return PS_OK;
}

int ps_planner_outlier_fits(double cycle, double now_in_cycle, double remaining_scheduled, double exec_time) {
  return (cycle - now_in_cycle) - remaining_scheduled >= exec_time - 1e-12 ? 1 : 0;
}

}  // extern "C"
