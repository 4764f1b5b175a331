// Drives the host-only planner (ps_planner_*) through a long seeded sequence of
// job arrivals, task assignments and job exits.  Built by the test suite together
// with ps_planner.cpp under AddressSanitizer and UndefinedBehaviorSanitizer: any
// out-of-bounds access, use after free, leak or undefined arithmetic in the
// planner aborts the run.  No device is involved.
#include <cstdio>
#include <cstdlib>
#include <vector>

#include "ps_b200.h"

static unsigned long long state = 0x9e3779b97f4a7c15ull;
static unsigned int next_u32() {
  state = state * 6364136223846793005ull + 1442695040888963407ull;
  return (unsigned int)(state >> 33);
}
static double uniform(double lo, double hi) { return lo + (hi - lo) * (next_u32() / 2147483648.0); }

#define CHECK(x)                                                            \
  do {                                                                      \
    if (!(x)) {                                                             \
      std::fprintf(stderr, "planner_sanitized: line %d: %s\n", __LINE__, #x); \
      return 1;                                                             \
    }                                                                       \
  } while (0)

int main() {
  for (int round = 0; round < 6; ++round) {
    ps_planner* pl = nullptr;
    CHECK(ps_planner_create(&pl, round % 2 ? 0.1 : 0.25) == PS_OK);
    std::vector<int> live;
    std::vector<int> tasks;
    for (int step = 0; step < 1500; ++step) {
      const unsigned int op = next_u32() % 100;
      if (live.empty() || op < 12) {
        int j = -1;
        CHECK(ps_planner_add_job(pl, uniform(2.0, 40.0), &j) == PS_OK && j >= 0);
        live.push_back(j);
      } else if (op < 90) {
        const int j = live[next_u32() % live.size()];
        int t = -1, a = -1;
        CHECK(ps_planner_assign(pl, j, uniform(0.01, 1.5), &t, &a) == PS_OK && t >= 0 && a >= 0);
        tasks.push_back(t);
        int runs = 0;
        double period = 0.0;
        CHECK(ps_planner_task_runs(pl, t, &runs, &period) == PS_OK && runs >= 1 && period > 0.0);
      } else if (live.size() > 1) {
        const size_t k = next_u32() % live.size();
        int released = -1;
        CHECK(ps_planner_remove_job(pl, live[k], &released) == PS_OK && released >= 0);
        live.erase(live.begin() + (long)k);
      }
      if (step % 97 == 0) {
        int allocated = 0, alive = 0;
        CHECK(ps_planner_num_aggregators(pl, &allocated, &alive) == PS_OK && alive <= allocated);
        for (int n = 0; n < allocated; ++n) {
          int is_alive = 0, nt = 0;
          double cycle = 0.0, load = 0.0;
          CHECK(ps_planner_aggregator_info(pl, n, &is_alive, &cycle, &load, &nt) == PS_OK);
          CHECK(load >= 0.0 && cycle >= 0.0 && nt >= 0 && (is_alive || nt == 0));
        }
        for (int j : live) {
          double profiled = 0.0, current = 0.0, loss = 0.0;
          CHECK(ps_planner_job_info(pl, j, &profiled, &current, &loss) == PS_OK && current >= profiled * (1 - 1e-9));
        }
      }
    }
    // calls that must be refused
    int dummy = 0;
    CHECK(ps_planner_assign(pl, 1 << 20, 1.0, &dummy, &dummy) == PS_ERR_BAD_ARG);
    CHECK(ps_planner_task_info(pl, -1, &dummy, &dummy, nullptr) == PS_ERR_BAD_ARG);
    CHECK(ps_planner_aggregator_info(pl, 1 << 20, &dummy, nullptr, nullptr, &dummy) == PS_ERR_BAD_ARG);
    CHECK(ps_planner_destroy(pl) == PS_OK);
  }
  CHECK(ps_planner_outlier_fits(12.0, 3.0, 2.0, 1.0) == 1);
  std::printf("planner_sanitized: ok\n");
  return 0;
}
