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

struct __align__(16) PsTaskDev {       // 128 bytes, one per ready (job, block)
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
  unsigned int chunk_elems;            // elements per chunk of THIS task (multiple of 1024, or of row_len)
  unsigned int row_len;                // > 0: some shards of this task are row-sparse; elements per row
  unsigned int sparse_row;             // index of the task's first PsSparseDev entry (one per worker)
  unsigned int _r2;
  // device-time profile of this task, filled only when the table asks for it
  unsigned long long busy_ns;          // sum over chunks of (chunk end - chunk start)      (uploaded as 0)
  unsigned long long t_first;          // earliest chunk start, %globaltimer ns             (uploaded as ~0)
  unsigned long long t_last;           // latest chunk end                                  (uploaded as 0)
  unsigned long long _r3;
};

struct __align__(16) PsTableHdr {      // 48 bytes at the start of the table
  unsigned int counter;                // next chunk to claim (uploaded as 0)
  unsigned int n_tasks;
  unsigned int total_chunks;
  unsigned int chunk_elems;            // largest chunk size used in this table
  unsigned int tasks_off, starts_off, ptrs_off;   // byte offsets from the table base
  unsigned int parts_per_chunk;        // partial sums each chunk publishes (1 per CTA or 1 per consumer warp)
  unsigned int profile;                // 1: record per-task device time (direct-load kernel)
  unsigned int sparse_off;             // byte offset of the PsSparseDev array (row-sparse shards)
  unsigned int exited;                 // CTAs that have left the launch (uploaded as 0)
  unsigned int wait_units;             // bulk-copy kernel: limit of every mbarrier wait, in units of 1024 cycles
};

// One worker's shard of a row-sparse task: the sorted ids of the rows it holds
// (block-local) — its values pointer sits in the ordinary shard-pointer row and
// points at n packed rows.  ids == nullptr: this worker pushed a dense shard.
struct __align__(16) PsSparseDev {
  const int* ids;
  unsigned int n;
  unsigned int _pad;
};

struct __align__(16) PsStat {          // 48 bytes per registered block, written by the task's last chunk
  double sqnorm;
  unsigned long long step;
  unsigned long long busy_ns, t_first, t_last;   // zero unless profiling was on
  unsigned long long _r0;
};

}  // namespace psb
