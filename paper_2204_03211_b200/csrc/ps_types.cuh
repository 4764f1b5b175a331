// Device-side data structures of the packed aggregation service.
//
// One launch serves any mix of jobs: the host uploads a task table — a header,
// one PsTaskDev per ready (job, block), the first chunk index of every task and
// the W shard pointers of every task — and persistent CTAs claim
// (job, block, chunk) work items from an atomic counter until the table is
// exhausted (paper Section 3.3: aggregation tasks of many jobs are packed onto
// one shared Aggregator; Section 2.2: tensors are independent, so chunks can be
// processed in any order by any CTA).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace psb {

constexpr int kMaxWorkers = 256;

struct __align__(16) PsJobDev {        // 64 bytes, one per registered job
  int opt, grad_dtype, W, _pad;
  float lr, mom, wd, b1, b2, omb1, omb2, eps, gs, _r0, _r1, _r2;
};

struct __align__(16) PsTaskDev {       // 96 bytes, one per ready (job, block)
  float* p;
  float* s0;
  float* s1;
  unsigned long long nelem;
  unsigned int shard_row;              // index of the task's first shard pointer
  unsigned int first_chunk;
  unsigned int nchunks;
  unsigned int ticket;                 // partial sums delivered so far (uploaded as 0)
  float ss_t, sbc2_t;                  // Adam step size and sqrt(1 - b2^t)
  int job;
  unsigned int stat_idx;
  unsigned long long step;
  unsigned int vec_ok;                 // all pointers 16-byte aligned
  unsigned int tile_elems;             // elements per ring tile (bulk-copy kernel); 0 = direct loads only
  unsigned int chunk_elems;            // elements per chunk of THIS task (multiple of 1024)
  unsigned int _r0, _r1, _r2;
};

struct __align__(16) PsTableHdr {      // 32 bytes at the start of the table
  unsigned int counter;                // next chunk to claim (uploaded as 0)
  unsigned int n_tasks;
  unsigned int total_chunks;
  unsigned int chunk_elems;            // largest chunk size used in this table
  unsigned int tasks_off, starts_off, ptrs_off;   // byte offsets from the table base
  unsigned int parts_per_chunk;        // partial sums each chunk publishes (1 per CTA or 1 per consumer warp)
};

struct __align__(16) PsStat {
  double sqnorm;
  unsigned long long step;
};

}  // namespace psb
