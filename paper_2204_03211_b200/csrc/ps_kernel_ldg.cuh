// Aggregation kernel, direct-load variant: persistent CTAs claim
// (job, block, chunk) work items from the table's atomic counter and read the
// gradient shards straight from global memory with 128-bit streaming loads.
// Handles every case (any W, any alignment).
#pragma once

#include "ps_math.cuh"
#include "ps_rows.cuh"

namespace psb {

constexpr int kThreads = 256;          // threads per CTA

__global__ void __launch_bounds__(kThreads, 4)
ps_aggregate_ldg_kernel(unsigned char* __restrict__ table, const PsJobDev* __restrict__ jobs,
                        PsStat* __restrict__ stats, double* __restrict__ partials,
                        unsigned long long* done_word, unsigned long long seq) {
  PsTableHdr* hdr = reinterpret_cast<PsTableHdr*>(table);
  PsTaskDev* tasks = reinterpret_cast<PsTaskDev*>(table + hdr->tasks_off);
  const unsigned int* starts = reinterpret_cast<const unsigned int*>(table + hdr->starts_off);
  const void* const* ptrs = reinterpret_cast<const void* const*>(table + hdr->ptrs_off);
  const PsSparseDev* sparse = reinterpret_cast<const PsSparseDev*>(table + hdr->sparse_off);
  const unsigned int n_tasks = hdr->n_tasks, total = hdr->total_chunks;
  const bool profile = hdr->profile != 0;

  __shared__ unsigned int s_idx[2];
  __shared__ unsigned int s_task;
  __shared__ double s_red[kThreads / 32];
  __shared__ const void* s_rowsrc[kThreads / 32][32];   // row-sparse tasks: a row's sources, per warp

  const unsigned int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  unsigned int cursor = 0;   // meaningful in warp 0
  int buf = 0;
  if (tid == 0) s_idx[0] = atomicAdd(&hdr->counter, 1u);
  __syncthreads();

  while (true) {
    const unsigned int idx = s_idx[buf];
    if (idx >= total) break;
    if (warp == 0) {
      cursor = find_task(starts, n_tasks, cursor, idx, lane);
      if (lane == 0) s_task = cursor;
    } else if (tid == kThreads - 1) {
      s_idx[buf ^ 1] = atomicAdd(&hdr->counter, 1u);   // the next claim overlaps this chunk
    }
    __syncthreads();

    const unsigned long long t_begin = (profile && tid == 0) ? global_ns() : 0ull;
    const unsigned int t = s_task;
    const PsTaskDev* T = tasks + t;
    const unsigned int chunk_elems = T->chunk_elems;
    const size_t begin = (size_t)(idx - T->first_chunk) * chunk_elems;
    const unsigned int count = (unsigned int)min((unsigned long long)chunk_elems, T->nelem - begin);
    double sq = 0.0;
    if (T->row_len)
      run_rows_any<kThreads>(tid, jobs + T->job, T, ptrs + T->shard_row, sparse + T->sparse_row, begin, count,
                             s_rowsrc[warp], sq);
    else
      run_chunk_any<kThreads>(tid, jobs + T->job, T, ptrs + T->shard_row, begin, count, sq);

    // chunk sum of squares: lanes, then warps, in a fixed order
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sq += __shfl_down_sync(0xffffffffu, sq, o);
    if (lane == 0) s_red[warp] = sq;
    __syncthreads();
    if (tid == 0) {
      double s = s_red[0];
#pragma unroll
      for (int k = 1; k < kThreads / 32; ++k) s += s_red[k];
      if (profile) profile_chunk(tasks + t, t_begin, global_ns());
      publish_one(tasks, t, idx, s, stats, partials);
    }
    buf ^= 1;
  }
  signal_exit(&hdr->exited, done_word, seq);
}

}  // namespace psb
