// Aggregation kernel for small launches: the task table travels in the kernel's
// parameter space instead of being uploaded, and every CTA owns exactly one
// chunk (grid = number of chunks), so there is no work counter either.  A round
// of a few small tensors then costs one launch and no copy: what bounds such
// rounds is per-launch latency, not bandwidth.  Same chunk bodies, same bits.
#pragma once

#include "ps_kernel_ldg.cuh"

namespace psb {

// The table has the layout of the uploaded one (header, tasks, chunk starts,
// shard pointers); with the other arguments it stays below the 4 KB that every
// driver accepts as kernel parameters.
constexpr unsigned int kInlineBytes = 3968;
struct __align__(16) PsInlineTable {
  unsigned char bytes[kInlineBytes];
};

// Mutable per-task state of an inline launch (the parameter space is read-only).
// All-zero between launches: the CTA that finalizes a task clears its entry.
struct __align__(16) PsTaskMut {
  unsigned int ticket;
  unsigned int _pad;
  unsigned long long busy_ns;
  unsigned long long t_first_c;         // complement of the earliest chunk start (so that zero means "none yet")
  unsigned long long t_last;
};
constexpr unsigned int kInlineMaxTasks = kInlineBytes / sizeof(PsTaskDev);

__global__ void __launch_bounds__(kThreads, 4)
ps_aggregate_inline_kernel(const __grid_constant__ PsInlineTable tbl, const PsJobDev* __restrict__ jobs,
                           PsStat* __restrict__ stats, double* __restrict__ partials, PsTaskMut* __restrict__ mut,
                           unsigned int* exit_ctr, unsigned long long* done_word, unsigned long long seq) {
  // The next launch of this stream may start its own prologue now; it waits (below, in
  // its own code) for this launch to complete before it touches any data.
  pdl_launch_dependents();
  const unsigned char* table = tbl.bytes;
  const PsTableHdr* hdr = reinterpret_cast<const PsTableHdr*>(table);
  const PsTaskDev* tasks = reinterpret_cast<const PsTaskDev*>(table + hdr->tasks_off);
  const unsigned int* starts = reinterpret_cast<const unsigned int*>(table + hdr->starts_off);
  const void* const* ptrs = reinterpret_cast<const void* const*>(table + hdr->ptrs_off);
  const unsigned int n_tasks = hdr->n_tasks;
  const bool profile = hdr->profile != 0;

  __shared__ double s_red[kThreads / 32];
  const unsigned int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const unsigned int idx = blockIdx.x;

  // the task that owns chunk idx: the last one whose first chunk is <= idx (every warp finds it for itself)
  unsigned int t = 0;
  for (unsigned int base = 1; base < n_tasks; base += 32) {
    const unsigned int probe = base + lane;
    const bool le = probe < n_tasks && starts[probe] <= idx;
    const unsigned int adv = __popc(__ballot_sync(0xffffffffu, le));
    t += adv;
    if (adv < 32) break;
  }
  const PsTaskDev* T = tasks + t;
  const unsigned int chunk_elems = T->chunk_elems;
  const size_t begin = (size_t)(idx - T->first_chunk) * chunk_elems;
  const unsigned int count = (unsigned int)min((unsigned long long)chunk_elems, T->nelem - begin);

  // the job's hyper-parameters never change after registration: their load is in flight
  // while this launch waits for the stream's previous one
  const JobView job = load_job(jobs + T->job, T);

  // Everything above read kernel parameters and registration-time data only.  From here
  // on the launch reads and writes memory that the stream's previous launch may still be
  // working on.
  pdl_wait();

  const unsigned long long t_begin = (profile && tid == 0) ? global_ns() : 0ull;
  double sq = 0.0;
  run_chunk_view<kThreads>(tid, job, T, ptrs + T->shard_row, begin, count, sq);

#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sq += __shfl_down_sync(0xffffffffu, sq, o);
  if (lane == 0) s_red[warp] = sq;
  __syncthreads();
  if (warp == 0) {
    const unsigned int n = T->nchunks;
    PsTaskMut* M = mut + t;
    double s = 0.0;
    unsigned long long t_end = 0ull;
    unsigned int done = 0;
    if (lane == 0) {
      s = s_red[0];
#pragma unroll
      for (int k = 1; k < kThreads / 32; ++k) s += s_red[k];
      t_end = profile ? global_ns() : 0ull;
      if (n > 1) {
        if (profile) {
          atomicAdd(&M->busy_ns, t_end - t_begin);
          atomicMax(&M->t_first_c, ~t_begin);
          atomicMax(&M->t_last, t_end);
        }
        __stcg(partials + idx, s);
        __threadfence();
        done = atomicAdd(&M->ticket, 1u);
        __threadfence();
      }
    }
    done = __shfl_sync(0xffffffffu, done, 0);
    if (n == 1) {                          // the only chunk of its task: nothing to wait for
      if (lane == 0) {
        PsStat st;
        st.sqnorm = s;
        st.step = T->step;
        st.busy_ns = t_end - t_begin;
        st.t_first = t_begin;
        st.t_last = t_end;
        st._r0 = 0;
        stats[T->stat_idx] = st;
      }
    } else if (done == n - 1) {
      // last chunk of the task to finish: add the partial sums in a fixed order
      const double tot = sum_partials_warp(partials + T->first_chunk, n, lane);
      if (lane == 0) {
        PsStat st;
        st.sqnorm = tot;
        st.step = T->step;
        st.busy_ns = __ldcg(&M->busy_ns);
        const unsigned long long tfc = __ldcg(&M->t_first_c);
        st.t_first = tfc ? ~tfc : 0ull;
        st.t_last = __ldcg(&M->t_last);
        st._r0 = 0;
        stats[T->stat_idx] = st;
        M->ticket = 0;
        M->busy_ns = 0;
        M->t_first_c = 0;
        M->t_last = 0;
      }
    }
  }
  signal_exit(exit_ctr, done_word, seq);
}

}  // namespace psb
