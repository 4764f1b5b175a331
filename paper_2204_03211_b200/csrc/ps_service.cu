// Host runtime and C ABI of the packed model-aggregation service
// (declarations and contracts: include/ps_b200.h).
//
// Host side = the Aggregator's bookkeeping: registry of jobs and blocks keyed
// by (job ID, block ID) (paper Appendix A), push counting per iteration (BSP,
// paper Figure 1), the block -> context map that stands for the Agents'
// mapping table (paper Section 3.1), migration with the not-before-the-copy
// rule (paper Appendix B), and the builder of the packed task table that one
// kernel launch consumes (paper Section 3.3: tasks of many jobs share one
// Aggregator).  Every arithmetic step runs in the kernels of ps_device.cuh;
// there is no host fallback.
#include "../../include/ps_b200.h"

#include <algorithm>
#include <chrono>
#include <thread>
#include <type_traits>
#include <cmath>
#include <cstdint>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <string>
#include <vector>

#include "arena.h"
#include "ps_device.cuh"

namespace psb {

constexpr uint32_t kMagic = 0x50534232u;   // "PSB2"
constexpr int kSlots = 16;                 // task tables in flight
constexpr int kInlineGridFactor = 4;         // an inline launch has at most this many CTAs per resident slot
constexpr int kWorkStreams = 8;             // overlap mode: launches rotate over this many streams
constexpr unsigned int kMaxChunk = 1u << 20;

struct Job {
  ps_job_desc d;
  std::vector<int> block_of_id;            // block id -> index into Service::blocks, -1 = none
  mutable unsigned long long bc_step = 0;  // step the cached Adam scalars belong to
  mutable float bc_ss = 0.f, bc_sbc2 = 0.f;
  char* stage_base = nullptr;              // staging region of the job's blocks for pushes from host memory
  size_t stage_bytes = 0;
  size_t grad_esize() const { return d.grad_dtype == PS_BF16 ? 2 : 4; }
  int nstate() const { return d.opt == PS_ADAM ? 2 : 1; }
};

struct Block {
  int job = 0, id = 0;
  size_t nelem = 0;
  int ctx = 0;
  size_t off = 0, bytes = 0;               // one arena range: p | s0 | s1
  size_t sec = 0;                          // byte stride between p, s0, s1
  unsigned long long step = 0;
  std::vector<const void*> pushed;         // W entries, nullptr = not pushed
  std::vector<const int*> row_ids;         // W entries, non-null = that push was row-sparse
  std::vector<unsigned int> row_cnt;       // W entries, rows in a row-sparse push
  unsigned int row_len = 0;                // row length of this iteration's row-sparse pushes (0 = none)
  int nsparse = 0;
  int npushed = 0;
  unsigned int stat_idx = 0;
  unsigned long long mark = 0;             // duplicate detection inside one ready list
  int mark_pos = 0;                        // position in the list being examined (with mark)
  bool queued = false;                     // ready and validated, waiting in the service's batch for the next launch
  int last_slot = -1;                      // slot of the last aggregate
  unsigned long long last_slot_gen = 0;
  int mig_batch = -1;                      // migration batch whose copy may still be in flight
  void* staging = nullptr;                 // device buffer for ps_push_host: W rows of staging_row bytes
  size_t staging_row = 0;
  bool staging_own = false;                // its own allocation (else a range of the job's staging region)
};

struct Ctx {
  char* base = nullptr;
  Arena arena;
};

struct PendingFree {                       // source range of a migration, released when its batch has landed
  int ctx;
  size_t off, bytes;
  int batch;
};

// One ps_migrate_block(s) call: its copies complete together, at `ev`.
struct MigBatch {
  cudaEvent_t ev = nullptr;
  bool pending = false;
  unsigned long long seen_call = 0;        // the event was last queried during this API call ...
  bool seen_ready = false;                 // ... with this answer
  unsigned long long waited_call = 0;      // a stream wait was issued during this API call ...
  cudaStream_t waited_stream = nullptr;    // ... on this stream
};

struct Slot {
  unsigned char* host = nullptr;           // pinned
  unsigned char* dev = nullptr;
  size_t cap = 0;
  double* partials = nullptr;
  size_t partial_cap = 0;
  PsTaskMut* mut = nullptr;                // per-task state of launches whose table travels as a kernel parameter
  cudaEvent_t done = nullptr;              // marks a point of `stream` at or after the slot's launch
  bool done_recorded = false;              // ... once it has been recorded (lazily for launches that signal)
  cudaEvent_t copied = nullptr;            // table upload finished (recorded on the copy stream)
  cudaEvent_t input = nullptr;             // overlap mode: the caller's stream at the time of the call
  bool inflight = false;
  unsigned long long gen = 0;
  unsigned long long seq = 0;              // number of the slot's launch (what its kernel stores when it has finished)
  bool signals = false;                    // the kernel stores seq to the slot's completion word
  cudaStream_t stream = nullptr;           // the stream the launch went to
  int work_stream = -1;                    // its index among the service's streams, -1 = a caller's stream
};

struct Plan {                              // one built task table (host copy)
  std::vector<unsigned char> bytes;
  std::vector<int> order;                  // block indices in table order
  unsigned int total_chunks = 0, chunk_elems = 0;
  bool has_sparse = false;                 // some task carries row-sparse shards (direct-load kernel only)
  unsigned long long algo_bytes = 0;       // algorithmic bytes of the launch (dense semantics)
};

enum { kVarLdg = 0, kVarInline = 1, kVarBulk = 2, kVariants = 3 };

// A round that recurs every iteration (ps_round_prepare): the caller's lists, what
// they resolve to, and the packed task table of the last run.
struct Prepared {
  bool live = false;
  std::vector<int> jobs, block_ids, workers;   // the pushes as given
  std::vector<const void*> ptrs;
  std::vector<ps_task> ready;
  unsigned int flags = 0;
  unsigned long long epoch = ~0ull;        // registry/layout/option state the fields below belong to
  std::vector<int> push_bi;                // block index of every push
  std::vector<int> idx;                    // block index of every ready task
  bool self_contained = false;             // the pushes are exactly the W shards of every ready block
  bool plan_ok = false;                    // `plan` can be reused after patching the step fields
  Plan plan;
};

}  // namespace psb

using namespace psb;

struct ps_service {
  uint32_t magic = kMagic;
  int device = PS_DEVICE_NONE;
  int num_sms = 148;
  std::mutex mu;
  std::vector<Ctx> ctxs;
  std::vector<Job> jobs;
  std::vector<Block> blocks;
  std::vector<PendingFree> pending_free;
  std::vector<MigBatch> batches;
  unsigned long long call_id = 0;          // counts API calls that order work (dedupes event queries/waits)
  PsJobDev* jobs_dev = nullptr;
  size_t jobs_dev_cap = 0;
  PsStat* stats_dev = nullptr;
  size_t stats_dev_cap = 0;
  Slot slots[kSlots];
  int next_slot = 0;
  unsigned long long gen = 0;              // ready-list generation
  long long opt_chunk = 0, opt_ctas = 0, opt_sort = 1, opt_kernel = 0, opt_profile = 0;
  int* status_dev = nullptr;               // error word written by kernels whose waits expired
  cudaStream_t copy_stream = nullptr;      // table uploads run here, beside the previous launch
  cudaStream_t work_streams[kWorkStreams] = {};   // overlap mode: launches rotate over these
  int next_work = 0;
  // overlap mode: per service stream, the slot of its latest launch and that launch's number,
  // and the number of the latest launch a caller's stream has joined (ps_join)
  int ws_last_slot[kWorkStreams] = {};
  unsigned long long ws_last_seq[kWorkStreams] = {}, ws_joined_seq[kWorkStreams] = {};
  long long opt_overlap = 0;
  long long opt_inline = 1;               // small launches carry their table as a kernel parameter
  long long opt_streams = 4;              // overlap mode: launches rotate over this many of the service's streams
  long long opt_pdl = 1;                  // small launches are launched with programmatic stream serialization
  int occ_ctas = 0;
  unsigned long long launches = 0;
  unsigned long long var_launches[kVariants] = {}, var_bytes[kVariants] = {};
  // completion words, one per slot, in page-locked host memory: the kernel of a slot's launch
  // stores the launch number there when its last CTA leaves
  volatile unsigned long long* done_host = nullptr;
  unsigned long long* done_dev = nullptr;  // the same words as the device addresses them
  unsigned int* exit_ctrs = nullptr;       // device, one CTA counter per slot (inline launches), all-zero between launches
  Plan plan;                               // scratch reused by every ps_aggregate
  std::vector<int> idx;                    // the same for the validated ready list
  std::vector<int> free_blocks;            // entries of `blocks` released by ps_unregister_block
  std::vector<Prepared> prepared;          // ps_round_prepare
  // Packing of rounds over time (PS_OPT_BATCH): ready tasks that are held back while
  // earlier launches are still running, to go out together in the next launch
  std::vector<int> batch;                  // block indices, in arrival order
  unsigned long long batch_chunks = 0;     // their size in chunks of kChunkAuto elements
  int batch_rounds = 0;                    // how many rounds filled it
  long long opt_batch = 1;
  long long opt_split = 1;                 // large sets of ready blocks go out as a few overlapping launches
  std::vector<int> part;                   // scratch of launch_in_parts
  long long opt_wait_cycles = 4000000000ll;   // bulk-copy kernel: limit of a wait inside the kernel (about 2 s)
  bool mig_large_ok = true;                // the 28 KB kernel-parameter form of the migration kernel is accepted
  unsigned long long epoch = 0;            // bumped by whatever can invalidate a prepared round's table:
                                           // migration, import, unregistration, options
  int last_grid = 0, last_block = 0;
  const char* last_kernel = "none";
  std::string cuda_err;
};

namespace {

#define PS_CUDA(svc, call)                                                            \
  do {                                                                                \
    cudaError_t e__ = (call);                                                         \
    if (e__ != cudaSuccess) {                                                         \
      (svc)->cuda_err = std::string(#call) + ": " + cudaGetErrorString(e__);          \
      return PS_ERR_CUDA;                                                             \
    }                                                                                 \
  } while (0)

bool alive(const ps_service* s) { return s && s->magic == kMagic; }
bool has_device(const ps_service* s) { return s->device >= 0; }

int flush_batch(ps_service* s);     // launches what the batch holds (no-op without a device or when empty)

int find_block(ps_service* s, int job, int block) {
  if (job < 0 || job >= (int)s->jobs.size() || block < 0) return -1;
  const Job& j = s->jobs[job];
  if (block >= (int)j.block_of_id.size()) return -1;
  return j.block_of_id[block];
}

float* blk_p(ps_service* s, const Block& b) { return reinterpret_cast<float*>(s->ctxs[b.ctx].base + b.off); }
float* blk_s0(ps_service* s, const Block& b) { return reinterpret_cast<float*>(s->ctxs[b.ctx].base + b.off + b.sec); }
float* blk_s1(ps_service* s, const Block& b) {
  return s->jobs[b.job].nstate() == 2 ? reinterpret_cast<float*>(s->ctxs[b.ctx].base + b.off + 2 * b.sec) : nullptr;
}

// Releases source ranges of finished migrations.  With wait = true blocks
// until every pending copy has completed.
// Has the batch's copy landed?  The event is queried at most once per API call.
// *ready_out = false also when the query itself failed (rc != PS_OK).
int batch_ready(ps_service* s, int batch, bool wait, bool* ready_out) {
  MigBatch& m = s->batches[batch];
  *ready_out = true;
  if (!m.pending) return PS_OK;
  if (!wait && m.seen_call == s->call_id) { *ready_out = m.seen_ready; return PS_OK; }
  cudaError_t q = wait ? cudaEventSynchronize(m.ev) : cudaEventQuery(m.ev);
  if (q != cudaSuccess && q != cudaErrorNotReady) {
    *ready_out = false;
    s->cuda_err = std::string("migration event: ") + cudaGetErrorString(q);
    return PS_ERR_CUDA;
  }
  m.seen_call = s->call_id;
  m.seen_ready = (q == cudaSuccess);
  if (m.seen_ready) m.pending = false;
  *ready_out = m.seen_ready;
  return PS_OK;
}

int reap_frees(ps_service* s, bool wait) {
  size_t keep = 0;
  for (size_t i = 0; i < s->pending_free.size(); ++i) {
    PendingFree& f = s->pending_free[i];
    bool ready = false;
    int rc = batch_ready(s, f.batch, wait, &ready);
    if (rc) return rc;
    if (ready) s->ctxs[f.ctx].arena.release(f.off, f.bytes);
    else s->pending_free[keep++] = f;
  }
  s->pending_free.resize(keep);
  return PS_OK;
}

// reap = false: the caller has just released what finished migrations left behind (a batch of
// many blocks does that once, not once per block: the list it walks is as long as the batch)
int arena_alloc(ps_service* s, int ctx, size_t bytes, size_t* off_out, bool reap = true) {
  if (reap && has_device(s)) {
    int rc = reap_frees(s, false);
    if (rc) return rc;
  }
  size_t off = s->ctxs[ctx].arena.alloc(bytes);
  if (off == Arena::kNone && has_device(s) && !s->pending_free.empty()) {
    int rc = reap_frees(s, true);
    if (rc) return rc;
    off = s->ctxs[ctx].arena.alloc(bytes);
  }
  if (off == Arena::kNone) return PS_ERR_NOMEM;
  *off_out = off;
  return PS_OK;
}

template <typename T>
int grow_dev(ps_service* s, T** buf, size_t* cap, size_t need, bool zero_new) {
  if (need <= *cap) return PS_OK;
  size_t ncap = *cap ? *cap : 64;
  while (ncap < need) ncap *= 2;
  T* nbuf = nullptr;
  PS_CUDA(s, cudaMalloc(&nbuf, ncap * sizeof(T)));
  PS_CUDA(s, cudaDeviceSynchronize());
  if (zero_new) PS_CUDA(s, cudaMemset(nbuf, 0, ncap * sizeof(T)));
  if (*buf) {
    PS_CUDA(s, cudaMemcpy(nbuf, *buf, *cap * sizeof(T), cudaMemcpyDeviceToDevice));
  }
  // device memsets and device-to-device copies may return before they have run, and
  // the service's streams do not synchronize with the default stream
  PS_CUDA(s, cudaStreamSynchronize(cudaStreamLegacy));
  if (*buf) PS_CUDA(s, cudaFree(*buf));
  *buf = nbuf;
  *cap = ncap;
  return PS_OK;
}

// Validates a ready list (no state change besides the duplicate marks) and
// returns the block indices in list order.
int validate_ready_ids(ps_service* s, const ps_task* ready, int n_ready, std::vector<int>* out) {
  if (n_ready < 0 || (n_ready > 0 && !ready)) return PS_ERR_BAD_ARG;
  const unsigned long long gen = ++s->gen;
  out->clear();
  out->reserve(n_ready);
  for (int i = 0; i < n_ready; ++i) {
    const int bi = find_block(s, ready[i].job, ready[i].block);
    if (bi < 0) return PS_ERR_BAD_ARG;
    Block& b = s->blocks[bi];
    if (b.mark == gen) return PS_ERR_DUPLICATE;
    b.mark = gen;
    out->push_back(bi);
  }
  // a listed block that still waits in the batch: its earlier aggregate goes out first
  for (int bi : *out)
    if (s->blocks[bi].queued) {
      int rc = flush_batch(s);
      if (rc) return rc;
      break;
    }
  return PS_OK;
}

int validate_ready(ps_service* s, const ps_task* ready, int n_ready, std::vector<int>* out) {
  int rc = validate_ready_ids(s, ready, n_ready, out);
  if (rc) return rc;
  for (int bi : *out) {
    const Block& b = s->blocks[bi];
    if (b.npushed != s->jobs[b.job].d.num_workers) return PS_ERR_NOT_READY;
  }
  return PS_OK;
}

size_t bytes_per_elem(const Job& j) { return (size_t)j.d.num_workers * j.grad_esize() + 8 * (1 + j.nstate()); }

// Kernel variants (PS_OPT_KERNEL): 1 direct loads, 2 bulk-copy ring.
// Automatic = 1: the two are level on large fp32 launches; direct loads are ahead on bf16
// gradients, on jobs with many tiny tensors, and cover row-sparse shards and profiling.
enum { kKernelLdg = 1, kKernelBulk = 2 };
int kernel_of(const ps_service* s) { return s->opt_kernel == 0 ? kKernelLdg : (int)s->opt_kernel; }
bool use_bulk(const ps_service* s) { return kernel_of(s) == kKernelBulk; }

int grid_cap(ps_service* s) {
  int per_sm;
  if (use_bulk(s)) per_sm = 1;   // one warp-specialised CTA owns an SM's shared memory
  else if (s->opt_ctas > 0) per_sm = (int)s->opt_ctas;
  else per_sm = s->occ_ctas > 0 ? s->occ_ctas : 3;
  return s->num_sms * per_sm;
}

// One "wave" of work for the packing and splitting rules, in chunks: what the direct-load
// kernel's resident CTAs take at once.  A CTA of the ring kernel has an SM to itself and
// streams as much as four of those, so its waves are counted in the same unit.
unsigned long long work_wave(ps_service* s) {
  return use_bulk(s) ? 4ull * (unsigned long long)s->num_sms : (unsigned long long)grid_cap(s);
}

// Automatic chunk size.  Measured on B200 (C2, C4 all-ready and C4 in bursty
// rounds): 8192 elements beats 2048/4096/16384 and beats shrinking the chunks
// toward the end of the table; the per-launch cost that remains (about 30 us)
// is launch latency, ramp-up and the last wave, not chunk bookkeeping.
constexpr unsigned int kChunkAuto = 8192, kChunkFloor = 1024;

// A launch with fewer chunks than resident CTAs leaves SMs idle while each busy
// CTA streams a whole chunk at single-CTA bandwidth (about 19 us for 8192
// elements, measured): such small launches get smaller chunks, halving as long
// as the chunks still fit ONE wave of resident CTAs or until the floor is
// reached.  One wave of CTAs with two or four vectors per thread beats two or
// four waves of CTAs with one: every CTA pays its fixed cost (start, task lookup,
// the latency of its first loads, the reduction of the norm, the ticket) once.
unsigned int auto_chunk(ps_service* s, const std::vector<int>& idx, int grid) {
  unsigned int ce = kChunkAuto;
  while (ce > kChunkFloor) {
    unsigned long long chunks = 0;
    for (int bi : idx) chunks += (s->blocks[bi].nelem + ce / 2 - 1) / (ce / 2);
    if (chunks > (unsigned long long)grid) break;
    ce >>= 1;
  }
  return ce;
}

// Elements per ring tile of the bulk-copy kernel (0 would mean: direct loads only).  A
// tile is cut along the workers, so any number of workers fits.
unsigned int tile_elems_for(const Job&) { return kRingTile; }

// The fields of a task that change from one aggregate of its block to the next.
void set_step_fields(const Job& j, const Block& b, PsTaskDev* t) {
  const unsigned long long step = b.step + 1;
  // Adam's bias-correction scalars (binary64 pow, rounded once); blocks of a job
  // mostly share their step, so the last pair is remembered per job.  SGD: unused.
  t->ss_t = 0.f;
  t->sbc2_t = 0.f;
  if (j.d.opt == PS_ADAM) {
    if (j.bc_step != step) {
      j.bc_step = step;
      j.bc_ss = (float)((double)j.d.lr / (1.0 - std::pow((double)j.d.beta1, (double)step)));
      j.bc_sbc2 = (float)std::sqrt(1.0 - std::pow((double)j.d.beta2, (double)step));
    }
    t->ss_t = j.bc_ss;
    t->sbc2_t = j.bc_sbc2;
  }
  t->step = step;
}

// Builds the task table for the validated blocks `idx`.
int build_plan(ps_service* s, const std::vector<int>& idx, Plan* plan) {
  const size_t n = idx.size();
  plan->order = idx;
  const bool fixed = s->opt_chunk > 0;
  const unsigned int ce = fixed ? (unsigned int)s->opt_chunk : auto_chunk(s, idx, grid_cap(s));
  plan->chunk_elems = ce;
  if (s->opt_sort) {
    // heaviest chunks first: the launch's tail is then made of light chunks
    std::stable_sort(plan->order.begin(), plan->order.end(), [&](int a, int b) {
      const Block& A = s->blocks[a];
      const Block& B = s->blocks[b];
      const size_t ca = std::min<size_t>(A.nelem, ce) * bytes_per_elem(s->jobs[A.job]);
      const size_t cb = std::min<size_t>(B.nelem, ce) * bytes_per_elem(s->jobs[B.job]);
      return ca > cb;
    });
  }
  size_t nptr = 0;
  for (int bi : plan->order) nptr += s->jobs[s->blocks[bi].job].d.num_workers;

  const size_t tasks_off = sizeof(PsTableHdr);
  const size_t starts_off = tasks_off + n * sizeof(PsTaskDev);
  const size_t ptrs_off = (starts_off + n * sizeof(unsigned int) + 15) / 16 * 16;
  size_t nsp = 0;                        // PsSparseDev entries: W per task that has a row-sparse push
  for (int bi : plan->order)
    if (s->blocks[bi].nsparse) nsp += s->jobs[s->blocks[bi].job].d.num_workers;
  const size_t sparse_off = (ptrs_off + nptr * sizeof(void*) + 15) / 16 * 16;
  plan->bytes.assign(sparse_off + nsp * sizeof(PsSparseDev), 0);
  PsSparseDev* sp = reinterpret_cast<PsSparseDev*>(plan->bytes.data() + sparse_off);
  size_t sp_row = 0;
  plan->has_sparse = nsp > 0;
  unsigned char* base = plan->bytes.data();
  PsTaskDev* tasks = reinterpret_cast<PsTaskDev*>(base + tasks_off);
  unsigned int* starts = reinterpret_cast<unsigned int*>(base + starts_off);
  const void** ptrs = reinterpret_cast<const void**>(base + ptrs_off);
  unsigned long long chunk = 0;
  size_t row = 0;
  for (size_t i = 0; i < n; ++i) {
    const Block& b = s->blocks[plan->order[i]];
    const Job& j = s->jobs[b.job];
    PsTaskDev& t = tasks[i];
    t.p = blk_p(s, b);
    t.s0 = blk_s0(s, b);
    t.s1 = blk_s1(s, b);
    t.nelem = b.nelem;
    t.shard_row = (unsigned int)row;
    t.first_chunk = (unsigned int)chunk;
    t.chunk_elems = ce;
    t.row_len = 0;
    t.sparse_row = 0;
    if (b.nsparse) {
      // chunks of a row-sparse task are whole rows, and four times the dense size:
      // every warp re-positions its cursors (a binary search per worker) per chunk
      t.row_len = b.row_len;
      t.chunk_elems = std::max(1u, (fixed ? ce : 4 * ce) / b.row_len) * b.row_len;
      t.sparse_row = (unsigned int)sp_row;
      for (int w = 0; w < j.d.num_workers; ++w) {
        sp[sp_row + w].ids = b.row_ids[w];
        sp[sp_row + w].n = b.row_cnt[w];
      }
      sp_row += j.d.num_workers;
    }
    t.nchunks = (unsigned int)((b.nelem + t.chunk_elems - 1) / t.chunk_elems);
    t.ticket = 0;
    t.busy_ns = 0;
    t.t_first = ~0ull;
    t.t_last = 0;
    set_step_fields(j, b, &t);
    t.job = b.job;
    t.stat_idx = b.stat_idx;
    unsigned int vec = 1;
    for (int w = 0; w < j.d.num_workers; ++w) {
      ptrs[row + w] = b.pushed[w];
      if (reinterpret_cast<uintptr_t>(b.pushed[w]) & 15u) vec = 0;
    }
    t.vec_ok = vec;
    t.tile_elems = tile_elems_for(j);
    starts[i] = t.first_chunk;
    row += j.d.num_workers;
    chunk += t.nchunks;
    if (chunk > 0xfffffff0ull) return PS_ERR_BAD_ARG;
  }
  plan->total_chunks = (unsigned int)chunk;
  plan->algo_bytes = 0;
  for (int bi : plan->order) plan->algo_bytes += s->blocks[bi].nelem * bytes_per_elem(s->jobs[s->blocks[bi].job]);
  PsTableHdr* h = reinterpret_cast<PsTableHdr*>(base);
  h->counter = 0;
  h->n_tasks = (unsigned int)n;
  h->total_chunks = plan->total_chunks;
  h->chunk_elems = ce;
  h->tasks_off = (unsigned int)tasks_off;
  h->starts_off = (unsigned int)starts_off;
  h->ptrs_off = (unsigned int)ptrs_off;
  h->parts_per_chunk = 1;
  h->profile = s->opt_profile ? 1u : 0u;
  h->sparse_off = (unsigned int)sparse_off;
  h->exited = 0;
  h->wait_units = (unsigned int)std::min<long long>(0xffffffffll, (s->opt_wait_cycles + kWaitUnit - 1) / kWaitUnit);
  return PS_OK;
}

// Has the slot's launch finished?  Launches that signal are checked by reading
// their completion word (no driver call); the others by querying their event.
bool slot_finished(ps_service* s, Slot& sl) {
  if (!sl.inflight) return true;
  const int i = (int)(&sl - s->slots);
  if (sl.signals && s->done_host[i] == sl.seq) { sl.inflight = false; return true; }
  if (sl.done_recorded && cudaEventQuery(sl.done) == cudaSuccess) { sl.inflight = false; return true; }
  return false;
}

// An event at or after the slot's launch exists on its stream after this call.
int ensure_done_event(ps_service* s, Slot& sl) {
  if (sl.done_recorded) return PS_OK;
  PS_CUDA(s, cudaEventRecord(sl.done, sl.stream));
  sl.done_recorded = true;
  return PS_OK;
}

// Blocks the host until the slot's launch has finished.  A launch that signals is
// waited for by polling its completion word: an event recorded now would sit behind
// everything enqueued on that stream since, and waiting for it would drain the whole
// queue instead of this one launch.  The poll is bounded; past the bound (a launch that
// is itself held up for seconds, e.g. behind a caller's event) the event takes over.
int wait_slot(ps_service* s, Slot& sl) {
  if (slot_finished(s, sl)) return PS_OK;
  if (sl.signals) {
    const int i = (int)(&sl - s->slots);
    const auto t0 = std::chrono::steady_clock::now();
    for (unsigned int spin = 1;; ++spin) {
      if (s->done_host[i] == sl.seq) { sl.inflight = false; return PS_OK; }
      if ((spin & 1023u) == 0) {
        if (std::chrono::steady_clock::now() - t0 > std::chrono::seconds(2)) break;
        std::this_thread::yield();
      }
    }
  }
  int rc = ensure_done_event(s, sl);
  if (rc) return rc;
  PS_CUDA(s, cudaEventSynchronize(sl.done));
  sl.inflight = false;
  return PS_OK;
}

int acquire_slot(ps_service* s, size_t table_bytes, size_t nchunks, Slot** out) {
  Slot& sl = s->slots[s->next_slot];
  int rc = wait_slot(s, sl);
  if (rc) return rc;
  if (!sl.done) PS_CUDA(s, cudaEventCreateWithFlags(&sl.done, cudaEventDisableTiming));
  if (!sl.copied) PS_CUDA(s, cudaEventCreateWithFlags(&sl.copied, cudaEventDisableTiming));
  if (!sl.input) PS_CUDA(s, cudaEventCreateWithFlags(&sl.input, cudaEventDisableTiming));
  if (table_bytes > sl.cap) {
    size_t ncap = std::max<size_t>(table_bytes * 2, 1 << 16);
    if (sl.host) PS_CUDA(s, cudaFreeHost(sl.host));
    if (sl.dev) PS_CUDA(s, cudaFree(sl.dev));
    sl.host = nullptr; sl.dev = nullptr; sl.cap = 0;
    PS_CUDA(s, cudaHostAlloc(&sl.host, ncap, cudaHostAllocDefault));
    PS_CUDA(s, cudaMalloc(&sl.dev, ncap));
    sl.cap = ncap;
  }
  if (nchunks > sl.partial_cap) {
    size_t ncap = std::max<size_t>(nchunks * 2, 1 << 12);
    if (sl.partials) PS_CUDA(s, cudaFree(sl.partials));
    sl.partials = nullptr; sl.partial_cap = 0;
    PS_CUDA(s, cudaMalloc(&sl.partials, ncap * sizeof(double)));
    sl.partial_cap = ncap;
  }
  if (!sl.mut) {
    PS_CUDA(s, cudaMalloc(&sl.mut, kInlineMaxTasks * sizeof(PsTaskMut)));
    PS_CUDA(s, cudaMemset(sl.mut, 0, kInlineMaxTasks * sizeof(PsTaskMut)));   // kept all-zero by the kernel
    PS_CUDA(s, cudaStreamSynchronize(cudaStreamLegacy));                      // before a service stream uses it
  }
  *out = &sl;
  return PS_OK;
}

// The slot of the block's last launch if that launch may still be running, else nullptr.
Slot* pending_slot(ps_service* s, Block& b) {
  if (b.last_slot < 0) return nullptr;
  Slot& sl = s->slots[b.last_slot];
  if (sl.gen != b.last_slot_gen || slot_finished(s, sl)) return nullptr;
  return &sl;
}

// Makes `stream` wait for everything enqueued so far that touches block b.
// `waited` (optional) collects the slots this call has already made `stream`
// wait for, so that a list of many blocks from one earlier launch costs one wait.
// A launch that went to `stream` itself needs no wait: stream order covers it.
int order_after_block(ps_service* s, Block& b, cudaStream_t stream, unsigned int* waited = nullptr) {
  if (Slot* sl = pending_slot(s, b)) {
    const unsigned int bit = 1u << (unsigned)b.last_slot;
    // (a caller's stream handle may have been destroyed and handed out again, so only
    // the service's own streams are trusted to be the same stream when the handles match)
    const bool same = sl->work_stream >= 0 && sl->stream == stream;
    if (!same && !(waited && (*waited & bit))) {
      int rc = ensure_done_event(s, *sl);
      if (rc) return rc;
      PS_CUDA(s, cudaStreamWaitEvent(stream, sl->done, 0));
    }
    if (waited) *waited |= bit;
  }
  if (b.mig_batch >= 0) {
    bool ready = false;
    int rc = batch_ready(s, b.mig_batch, false, &ready);
    if (rc) return rc;
    if (ready) {
      b.mig_batch = -1;
    } else {
      MigBatch& m = s->batches[b.mig_batch];
      if (!(m.waited_call == s->call_id && m.waited_stream == stream)) {
        PS_CUDA(s, cudaStreamWaitEvent(stream, m.ev, 0));
        m.waited_call = s->call_id;
        m.waited_stream = stream;
      }
    }
  }
  return PS_OK;
}

// in_place: the kernel will read `ptr` itself (false: ps_push_host copies it to aligned staging first)
int push_checked(ps_service* s, int job, int block, int worker, const void* ptr, Block** out, bool in_place = true) {
  const int bi = find_block(s, job, block);
  if (bi < 0 || !ptr) return PS_ERR_BAD_ARG;
  Block& b = s->blocks[bi];
  const Job& j = s->jobs[b.job];
  if (worker < 0 || worker >= j.d.num_workers) return PS_ERR_BAD_ARG;
  if (reinterpret_cast<uintptr_t>(ptr) & (j.grad_esize() - 1)) return PS_ERR_ALIGN;
  if (b.queued) {                          // the pushes of its previous iteration are still held in the batch
    int rc = flush_batch(s);
    if (rc) return rc;
  }
  // a block with row-sparse pushes is streamed row by row with 128-bit loads from
  // every shard, the dense ones included: those need 16-byte aligned starts
  if (in_place && b.nsparse > 0 && (reinterpret_cast<uintptr_t>(ptr) & 15u)) return PS_ERR_ALIGN;
  if (b.pushed[worker]) return PS_ERR_DUPLICATE;
  *out = &b;
  return PS_OK;
}

// Launches one aggregation kernel with an optional programmatic-serialization attribute.
template <typename... KArgs, typename... Args>
cudaError_t launch_kernel(void (*kernel)(KArgs...), int grid, int block, size_t smem, cudaStream_t stream,
                                 bool pdl, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3((unsigned)block);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

}  // namespace

extern "C" {

int ps_create(ps_service** out, int device, int num_contexts, size_t arena_bytes_per_ctx) {
  if (!out || num_contexts < 1 || num_contexts > 1024 || device < PS_DEVICE_NONE) return PS_ERR_BAD_ARG;
  *out = nullptr;
  ps_service* s = new (std::nothrow) ps_service();
  if (!s) return PS_ERR_NOMEM;
  s->device = device;
  s->ctxs.resize(num_contexts);
  for (auto& c : s->ctxs) c.arena.reset(arena_bytes_per_ctx);
  if (device >= 0) {
    cudaError_t e = cudaSetDevice(device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&s->num_sms, cudaDevAttrMultiProcessorCount, device);
    if (e == cudaSuccess)
      e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&s->occ_ctas, ps_aggregate_ldg_kernel, kThreads, 0);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(ps_aggregate_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kBulkSmemBytes);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&s->copy_stream, cudaStreamNonBlocking);
    for (int i = 0; i < kWorkStreams && e == cudaSuccess; ++i)
      e = cudaStreamCreateWithFlags(&s->work_streams[i], cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaMalloc(&s->status_dev, sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(s->status_dev, 0, sizeof(int));
    if (e == cudaSuccess) e = cudaMalloc(&s->exit_ctrs, kSlots * sizeof(unsigned int));
    if (e == cudaSuccess) e = cudaMemset(s->exit_ctrs, 0, kSlots * sizeof(unsigned int));
    if (e == cudaSuccess) {
      void* h = nullptr;
      e = cudaHostAlloc(&h, kSlots * sizeof(unsigned long long), cudaHostAllocMapped);
      if (e == cudaSuccess) {
        std::memset(h, 0, kSlots * sizeof(unsigned long long));
        s->done_host = static_cast<volatile unsigned long long*>(h);
        void* d = nullptr;
        e = cudaHostGetDevicePointer(&d, h, 0);
        s->done_dev = static_cast<unsigned long long*>(d);
      }
    }
    if (e == cudaSuccess) e = cudaStreamSynchronize(cudaStreamLegacy);
    for (int c = 0; e == cudaSuccess && c < num_contexts; ++c) {
      void* base = nullptr;
      e = cudaMalloc(&base, s->ctxs[c].arena.capacity() ? s->ctxs[c].arena.capacity() : Arena::kAlign);
      s->ctxs[c].base = static_cast<char*>(base);
    }
    if (e != cudaSuccess) {
      const bool oom = (e == cudaErrorMemoryAllocation);
      for (auto& c : s->ctxs) if (c.base) cudaFree(c.base);
      if (s->status_dev) cudaFree(s->status_dev);
      if (s->exit_ctrs) cudaFree(s->exit_ctrs);
      if (s->done_host) cudaFreeHost(const_cast<unsigned long long*>(s->done_host));
      if (s->copy_stream) cudaStreamDestroy(s->copy_stream);
      for (auto ws : s->work_streams) if (ws) cudaStreamDestroy(ws);
      cudaGetLastError();
      delete s;
      return oom ? PS_ERR_NOMEM : PS_ERR_CUDA;
    }
  }
  *out = s;
  return PS_OK;
}

int ps_destroy(ps_service* s) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  if (has_device(s)) {
    cudaSetDevice(s->device);
    flush_batch(s);
    cudaDeviceSynchronize();
    for (auto& b : s->blocks)
      if (b.staging && b.staging_own) cudaFree(b.staging);
    for (auto& j : s->jobs)
      if (j.stage_base) cudaFree(j.stage_base);
    for (auto& m : s->batches)
      if (m.ev) cudaEventDestroy(m.ev);
    for (auto& sl : s->slots) {
      if (sl.host) cudaFreeHost(sl.host);
      if (sl.dev) cudaFree(sl.dev);
      if (sl.partials) cudaFree(sl.partials);
      if (sl.mut) cudaFree(sl.mut);
      if (sl.done) cudaEventDestroy(sl.done);
      if (sl.copied) cudaEventDestroy(sl.copied);
      if (sl.input) cudaEventDestroy(sl.input);
    }
    for (auto& c : s->ctxs) if (c.base) cudaFree(c.base);
    if (s->jobs_dev) cudaFree(s->jobs_dev);
    if (s->stats_dev) cudaFree(s->stats_dev);
    if (s->status_dev) cudaFree(s->status_dev);
    if (s->exit_ctrs) cudaFree(s->exit_ctrs);
    if (s->done_host) cudaFreeHost(const_cast<unsigned long long*>(s->done_host));
    if (s->copy_stream) cudaStreamDestroy(s->copy_stream);
    for (auto ws : s->work_streams) if (ws) cudaStreamDestroy(ws);
  }
  s->magic = 0;
  delete s;
  return PS_OK;
}

int ps_register_job(ps_service* s, const ps_job_desc* d, int* job_out) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  if (!d || !job_out) return PS_ERR_BAD_ARG;
  if (d->opt != PS_SGD && d->opt != PS_ADAM) return PS_ERR_BAD_ARG;
  if (d->grad_dtype != PS_F32 && d->grad_dtype != PS_BF16) return PS_ERR_BAD_ARG;
  if (d->num_workers < 1 || d->num_workers > PS_MAX_WORKERS) return PS_ERR_BAD_ARG;
  const int id = (int)s->jobs.size();
  if (has_device(s)) {
    PS_CUDA(s, cudaSetDevice(s->device));
    int rc = grow_dev(s, &s->jobs_dev, &s->jobs_dev_cap, (size_t)id + 1, false);
    if (rc) return rc;
    PsJobDev jd;
    std::memset(&jd, 0, sizeof jd);
    jd.opt = d->opt; jd.grad_dtype = d->grad_dtype; jd.W = d->num_workers;
    jd.lr = d->lr; jd.mom = d->momentum; jd.wd = d->weight_decay;
    jd.b1 = d->beta1; jd.b2 = d->beta2;
    jd.omb1 = 1.0f - d->beta1;
    jd.omb2 = 1.0f - d->beta2;
    jd.eps = d->eps; jd.gs = d->grad_scale;
    PS_CUDA(s, cudaMemcpy(s->jobs_dev + id, &jd, sizeof jd, cudaMemcpyHostToDevice));
    PS_CUDA(s, cudaStreamSynchronize(cudaStreamLegacy));   // a small pageable copy may still be in flight on return
  }
  Job j;
  j.d = *d;
  s->jobs.push_back(j);
  *job_out = id;
  return PS_OK;
}

int ps_register_block(ps_service* s, int job, int block, size_t nelem, int ctx, const float* init) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  if (job < 0 || job >= (int)s->jobs.size() || block < 0 || block >= (1 << 26)) return PS_ERR_BAD_ARG;
  if (nelem == 0 || nelem > ((size_t)1 << 40) || ctx < 0 || ctx >= (int)s->ctxs.size()) return PS_ERR_BAD_ARG;
  Job& j = s->jobs[job];
  if (block < (int)j.block_of_id.size() && j.block_of_id[block] >= 0) return PS_ERR_DUPLICATE;
  Block b;
  b.job = job; b.id = block; b.nelem = nelem; b.ctx = ctx;
  b.sec = Arena::round_up(nelem * sizeof(float));
  b.bytes = b.sec * (1 + j.nstate());
  b.pushed.assign(j.d.num_workers, nullptr);
  b.row_ids.assign(j.d.num_workers, nullptr);
  b.row_cnt.assign(j.d.num_workers, 0);
  // an entry released by ps_unregister_block is used again (with its statistics record), so
  // blocks that come and go, e.g. by migration between services, do not grow the tables
  const bool reuse = !s->free_blocks.empty();
  const size_t bi_new = reuse ? (size_t)s->free_blocks.back() : s->blocks.size();
  b.stat_idx = (unsigned int)bi_new;
  if (has_device(s)) PS_CUDA(s, cudaSetDevice(s->device));
  int rc = arena_alloc(s, ctx, b.bytes, &b.off);
  if (rc) return rc;
  if (has_device(s)) {
    rc = grow_dev(s, &s->stats_dev, &s->stats_dev_cap, bi_new + 1, true);
    cudaError_t e = cudaSuccess;
    if (!rc) {
      char* base = s->ctxs[ctx].base + b.off;
      e = cudaMemset(base, 0, b.bytes);
      if (e == cudaSuccess && reuse) e = cudaMemset(s->stats_dev + bi_new, 0, sizeof(PsStat));
      if (e == cudaSuccess && init) e = cudaMemcpy(base, init, nelem * sizeof(float), cudaMemcpyDefault);
      // a device memset may return before it has run, and the service's streams do not
      // synchronize with the default stream: wait here, once per registration
      if (e == cudaSuccess) e = cudaStreamSynchronize(cudaStreamLegacy);
      if (e != cudaSuccess) { s->cuda_err = cudaGetErrorString(e); rc = PS_ERR_CUDA; }
    }
    if (rc) { s->ctxs[ctx].arena.release(b.off, b.bytes); return rc; }
  }
  if (block >= (int)j.block_of_id.size()) j.block_of_id.resize(block + 1, -1);
  j.block_of_id[block] = (int)bi_new;
  if (reuse) {
    s->free_blocks.pop_back();
    s->blocks[bi_new] = std::move(b);
  } else {
    s->blocks.push_back(std::move(b));
  }
  return PS_OK;
}

int ps_push(ps_service* s, int job, int block, int worker, const void* ptr) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  Block* b = nullptr;
  int rc = push_checked(s, job, block, worker, ptr, &b);
  if (rc) return rc;
  b->pushed[worker] = ptr;
  b->npushed++;
  return PS_OK;
}

static int push_rows_locked(ps_service* s, int job, int block, int worker, const int* row_ids, int n_rows,
                            int row_len, const void* values);

int ps_push_rows(ps_service* s, int job, int block, int worker, const int* row_ids, int n_rows, int row_len,
                 const void* values) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  return push_rows_locked(s, job, block, worker, row_ids, n_rows, row_len, values);
}

int ps_push_rows_batch(ps_service* s, int n, const int* jobs, const int* blocks, const int* workers,
                       const int* const* row_ids, const int* n_rows, const int* row_lens,
                       const void* const* values) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  if (n < 0 || (n > 0 && (!jobs || !blocks || !workers || !row_ids || !n_rows || !row_lens || !values)))
    return PS_ERR_BAD_ARG;
  int rc = PS_OK, done = 0;
  for (; done < n; ++done) {
    rc = push_rows_locked(s, jobs[done], blocks[done], workers[done], row_ids[done], n_rows[done], row_lens[done],
                          values[done]);
    if (rc) break;
  }
  if (rc) {   // roll back: all-or-nothing
    for (int i = 0; i < done; ++i) {
      Block& b = s->blocks[find_block(s, jobs[i], blocks[i])];
      b.pushed[workers[i]] = nullptr;
      b.row_ids[workers[i]] = nullptr;
      b.row_cnt[workers[i]] = 0;
      b.npushed--;
      if (--b.nsparse == 0) b.row_len = 0;
    }
  }
  return rc;
}

static int push_rows_locked(ps_service* s, int job, int block, int worker, const int* row_ids, int n_rows,
                            int row_len, const void* values) {
  const int bi = find_block(s, job, block);
  if (bi < 0 || !row_ids || !values || n_rows < 0 || row_len <= 0) return PS_ERR_BAD_ARG;
  Block& b = s->blocks[bi];
  const Job& j = s->jobs[b.job];
  if (worker < 0 || worker >= j.d.num_workers || j.d.num_workers > kRowsMaxWorkers) return PS_ERR_BAD_ARG;
  if (b.nelem % (size_t)row_len != 0 || (size_t)n_rows > b.nelem / (size_t)row_len) return PS_ERR_BAD_ARG;
  if (b.row_len != 0 && b.row_len != (unsigned int)row_len) return PS_ERR_BAD_ARG;
  // rows are streamed with 128-bit accesses: whole vectors per row, aligned starts
  if (((size_t)row_len * j.grad_esize()) % 16 != 0 || (reinterpret_cast<uintptr_t>(values) & 15u) ||
      (reinterpret_cast<uintptr_t>(row_ids) & 3u))
    return PS_ERR_ALIGN;
  if (b.queued) {
    int rc = flush_batch(s);
    if (rc) return rc;
  }
  if (b.pushed[worker]) return PS_ERR_DUPLICATE;
  // the dense shards this block already holds will be read with 128-bit loads too
  for (int w = 0; w < j.d.num_workers; ++w)
    if (b.pushed[w] && !b.row_ids[w] && (reinterpret_cast<uintptr_t>(b.pushed[w]) & 15u)) return PS_ERR_ALIGN;
  b.pushed[worker] = values;
  b.row_ids[worker] = row_ids;
  b.row_cnt[worker] = (unsigned int)n_rows;
  b.row_len = (unsigned int)row_len;
  b.nsparse++;
  b.npushed++;
  return PS_OK;
}

static void unpush_locked(ps_service* s, int n, const int* jobs, const int* blocks, const int* workers) {
  for (int i = 0; i < n; ++i) {
    Block& b = s->blocks[find_block(s, jobs[i], blocks[i])];
    b.pushed[workers[i]] = nullptr;
    b.npushed--;
  }
}

static int push_batch_locked(ps_service* s, int n, const int* jobs, const int* blocks, const int* workers,
                             const void* const* ptrs) {
  if (n < 0 || (n > 0 && (!jobs || !blocks || !workers || !ptrs))) return PS_ERR_BAD_ARG;
  int rc = PS_OK, done = 0;
  for (; done < n; ++done) {
    Block* b = nullptr;
    rc = push_checked(s, jobs[done], blocks[done], workers[done], ptrs[done], &b);
    if (rc) break;
    b->pushed[workers[done]] = ptrs[done];
    b->npushed++;
  }
  if (rc) unpush_locked(s, done, jobs, blocks, workers);   // all-or-nothing
  return rc;
}

int ps_push_batch(ps_service* s, int n, const int* jobs, const int* blocks, const int* workers,
                  const void* const* ptrs) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  return push_batch_locked(s, n, jobs, blocks, workers, ptrs);
}

// Gives block b a staging buffer for pushes from host memory.  The first such push
// of a job allocates ONE region for all blocks the job has then, laid out block after
// block in id order, each block W rows of round_up(nelem * element size, 256) bytes:
// shards that are neighbours in the caller's host buffer in that same layout are then
// neighbours on the device too and travel as one copy.  Blocks registered later get
// an allocation of their own.
static int ensure_staging(ps_service* s, Block& b) {
  if (b.staging) return PS_OK;
  Job& j = s->jobs[b.job];
  const size_t W = (size_t)j.d.num_workers;
  if (!j.stage_base) {
    size_t total = 0;
    for (int bi : j.block_of_id)
      if (bi >= 0) total += Arena::round_up(s->blocks[bi].nelem * j.grad_esize()) * W;
    void* base = nullptr;
    cudaError_t e = cudaMalloc(&base, total ? total : 256);
    if (e != cudaSuccess) {
      cudaGetLastError();
      if (e == cudaErrorMemoryAllocation) return PS_ERR_NOMEM;
      s->cuda_err = cudaGetErrorString(e);
      return PS_ERR_CUDA;
    }
    j.stage_base = static_cast<char*>(base);
    j.stage_bytes = total;
    size_t off = 0;
    for (int bi : j.block_of_id) {
      if (bi < 0) continue;
      Block& o = s->blocks[bi];
      if (o.staging) continue;             // (keeps an allocation of its own)
      o.staging_row = Arena::round_up(o.nelem * j.grad_esize());
      o.staging = j.stage_base + off;
      o.staging_own = false;
      off += o.staging_row * W;
    }
    if (b.staging) return PS_OK;
  }
  b.staging_row = Arena::round_up(b.nelem * j.grad_esize());
  cudaError_t e = cudaMalloc(&b.staging, b.staging_row * W);
  if (e != cudaSuccess) {
    b.staging = nullptr;
    cudaGetLastError();
    if (e == cudaErrorMemoryAllocation) return PS_ERR_NOMEM;
    s->cuda_err = cudaGetErrorString(e);
    return PS_ERR_CUDA;
  }
  b.staging_own = true;
  return PS_OK;
}

int ps_push_host_batch(ps_service* s, int n, const int* jobs, const int* blocks, const int* workers,
                       const void* const* host_ptrs, void* stream_) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  if (n < 0 || (n > 0 && (!jobs || !blocks || !workers || !host_ptrs))) return PS_ERR_BAD_ARG;
  // validation first: nothing is copied or recorded unless every entry is acceptable
  std::vector<Block*> bs((size_t)n);
  const unsigned long long gen = ++s->gen;
  for (int i = 0; i < n; ++i) {
    int rc = push_checked(s, jobs[i], blocks[i], workers[i], host_ptrs[i], &bs[i], false);
    if (rc) return rc;
  }
  {                                        // the same (block, worker) twice in one batch
    std::vector<unsigned char> seen;
    for (int i = 0; i < n; ++i) {
      Block& b = *bs[i];
      if (b.mark != gen) { b.mark = gen; b.mark_pos = (int)seen.size(); seen.resize(seen.size() + b.pushed.size(), 0); }
      unsigned char& f = seen[(size_t)b.mark_pos + (size_t)workers[i]];
      if (f) return PS_ERR_DUPLICATE;
      f = 1;
    }
  }
  if (!has_device(s)) return PS_ERR_NO_DEVICE;
  if (n == 0) return PS_OK;
  PS_CUDA(s, cudaSetDevice(s->device));
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  for (int i = 0; i < n; ++i) {
    int rc = ensure_staging(s, *bs[i]);
    if (rc) return rc;
  }
  // the staging rows may still be read by the blocks' previous aggregates
  ++s->call_id;
  unsigned int waited = 0;
  for (int i = 0; i < n; ++i) {
    if (i && bs[i] == bs[i - 1]) continue;
    int rc = order_after_block(s, *bs[i], stream, &waited);
    if (rc) return rc;
  }
  // copies: neighbours on both sides are merged (the padding between rows travels with them)
  struct Range { char* dst; const char* src; size_t bytes; size_t span; };
  std::vector<Range> rs((size_t)n);
  for (int i = 0; i < n; ++i) {
    Block& b = *bs[i];
    rs[i].dst = static_cast<char*>(b.staging) + (size_t)workers[i] * b.staging_row;
    rs[i].src = static_cast<const char*>(host_ptrs[i]);
    rs[i].bytes = b.nelem * s->jobs[b.job].grad_esize();
    rs[i].span = b.staging_row;
  }
  std::vector<int> order((size_t)n);
  for (int i = 0; i < n; ++i) order[i] = i;
  std::sort(order.begin(), order.end(), [&](int a, int b) { return rs[a].dst < rs[b].dst; });
  for (size_t k = 0; k < order.size();) {
    const Range& first = rs[order[k]];
    size_t len = first.bytes, span = first.span, m = k + 1;
    while (m < order.size() && rs[order[m]].dst == first.dst + span && rs[order[m]].src == first.src + span) {
      len = span + rs[order[m]].bytes;
      span += rs[order[m]].span;
      ++m;
    }
    PS_CUDA(s, cudaMemcpyAsync(first.dst, first.src, len, cudaMemcpyHostToDevice, stream));
    k = m;
  }
  for (int i = 0; i < n; ++i) {
    bs[i]->pushed[workers[i]] = rs[i].dst;
    bs[i]->npushed++;
  }
  return PS_OK;
}

int ps_push_host(ps_service* s, int job, int block, int worker, const void* host_ptr, void* stream) {
  return ps_push_host_batch(s, 1, &job, &block, &worker, &host_ptr, stream);
}

static int launch_plan(ps_service* s, const std::vector<int>& idx, Plan& plan, cudaStream_t stream,
                       unsigned int flags);

// Launches the kernel for a built task table `plan` of the blocks `idx` (device current).
static int launch_plan(ps_service* s, const std::vector<int>& idx, Plan& plan, cudaStream_t stream,
                       unsigned int flags) {
  ++s->call_id;
  int rc = PS_OK;
  Slot* sl = nullptr;
  const bool bulk = use_bulk(s) && !plan.has_sparse;
  // A small table (a round of a few tensors) travels as a kernel parameter: no
  // upload, no copy event, and one CTA per chunk instead of a work counter.
  const bool inl = s->opt_inline && !bulk && !plan.has_sparse && plan.bytes.size() <= kInlineBytes &&
                   plan.total_chunks <= (unsigned int)(kInlineGridFactor * grid_cap(s));
  rc = acquire_slot(s, inl ? 0 : plan.bytes.size(),
                    (size_t)plan.total_chunks, &sl);
  if (rc) return rc;
  const int slot_index = (int)(sl - s->slots);
  // Overlap mode: the launch goes to one of the service-owned streams, after the
  // work the caller has enqueued on `stream` so far; consecutive launches then
  // overlap (the next one's CTAs fill the SMs the previous one's tail leaves idle).
  // A launch that has to follow an unfinished one (a block aggregated again) goes to
  // that launch's stream, where stream order is the dependency: no event.
  cudaStream_t run = stream;
  int ws = -1;
  if (s->opt_overlap) {
    // (small launches only: there the two driver calls of an event dependency are what a
    // launch costs.  A large launch takes the next stream and waits for exactly the launches
    // it depends on — behind its predecessor's stream it would also wait for whatever else
    // has been enqueued there since.)
    if (inl)
      for (int bi : idx) {
        Slot* dep = pending_slot(s, s->blocks[bi]);
        if (dep && dep->work_stream >= 0) { ws = dep->work_stream; break; }
      }
    if (ws < 0) {
      ws = s->next_work;
      s->next_work = (s->next_work + 1) % (int)s->opt_streams;
    }
    run = s->work_streams[ws];
    if (!(flags & PS_ROUND_INPUTS_COMPLETE)) {
      PS_CUDA(s, cudaEventRecord(sl->input, stream));
      PS_CUDA(s, cudaStreamWaitEvent(run, sl->input, 0));
    }
  }
  unsigned int waited = 0;
  for (int bi : idx) {
    rc = order_after_block(s, s->blocks[bi], run, &waited);
    if (rc) return rc;
  }
  const unsigned long long seq = s->launches + 1;
  unsigned long long* done_word = s->done_dev + slot_index;
  int grid = (int)std::min<unsigned long long>(plan.total_chunks, (unsigned long long)grid_cap(s));
  cudaError_t le;
  if (inl) {
    PsInlineTable tbl;
    std::memcpy(tbl.bytes, plan.bytes.data(), plan.bytes.size());
    grid = (int)plan.total_chunks;
    le = launch_kernel(ps_aggregate_inline_kernel, grid, kThreads, 0, run, s->opt_pdl != 0, tbl,
                       (const PsJobDev*)s->jobs_dev, s->stats_dev, sl->partials, sl->mut, s->exit_ctrs + slot_index,
                       done_word, seq);
  } else {
    std::memcpy(sl->host, plan.bytes.data(), plan.bytes.size());
    // The table depends on nothing the caller enqueued, so its upload goes to the
    // service's own stream and overlaps the previous launch; the kernel waits for it.
    PS_CUDA(s, cudaMemcpyAsync(sl->dev, sl->host, plan.bytes.size(), cudaMemcpyHostToDevice, s->copy_stream));
    PS_CUDA(s, cudaEventRecord(sl->copied, s->copy_stream));
    PS_CUDA(s, cudaStreamWaitEvent(run, sl->copied, 0));
    if (bulk)
      le = launch_kernel(ps_aggregate_bulk_kernel, grid, kBulkThreads, kBulkSmemBytes, run, false, sl->dev,
                         (const PsJobDev*)s->jobs_dev, s->stats_dev, sl->partials, s->status_dev, done_word, seq);
    else
      le = launch_kernel(ps_aggregate_ldg_kernel, grid, kThreads, 0, run, false, sl->dev,
                         (const PsJobDev*)s->jobs_dev, s->stats_dev, sl->partials, done_word, seq);
  }
  if (le != cudaSuccess) {
    s->cuda_err = std::string("kernel launch: ") + cudaGetErrorString(le);
    cudaGetLastError();
    return PS_ERR_CUDA;
  }
  sl->seq = seq;
  sl->gen = seq;                           // what a block remembers of its last launch (unique per launch)
  sl->signals = true;
  sl->stream = run;
  sl->work_stream = ws;
  sl->done_recorded = false;
  sl->inflight = true;
  // Every launch is marked by an event at once.  (Marking small launches only when another
  // stream had to wait for them saved a driver call per launch, but without the records
  // launches on different streams stopped overlapping reliably — measured: a replay of 54
  // small rounds took 0.32 to 0.49 ms from run to run, against a steady 0.40 ms with the
  // records.  Completion is still learnt from the kernels' completion words where the host
  // only needs to know, not to order streams.)
  PS_CUDA(s, cudaEventRecord(sl->done, run));
  sl->done_recorded = true;
  if (ws >= 0) {
    s->ws_last_slot[ws] = slot_index;
    s->ws_last_seq[ws] = seq;
  }
  s->next_slot = (s->next_slot + 1) % kSlots;
  s->launches = seq;
  const int var = inl ? kVarInline : bulk ? kVarBulk : kVarLdg;
  s->var_launches[var]++;
  s->var_bytes[var] += plan.algo_bytes;
  s->last_grid = grid;
  s->last_block = bulk ? kBulkThreads : kThreads;
  s->last_kernel = inl ? "inline" : bulk ? "bulk" : "ldg";
  for (int bi : idx) {
    Block& b = s->blocks[bi];
    b.step++;
    std::fill(b.pushed.begin(), b.pushed.end(), nullptr);
    std::fill(b.row_ids.begin(), b.row_ids.end(), nullptr);
    std::fill(b.row_cnt.begin(), b.row_cnt.end(), 0u);
    b.row_len = 0;
    b.nsparse = 0;
    b.npushed = 0;
    b.last_slot = slot_index;
    b.last_slot_gen = sl->gen;
  }
  return PS_OK;
}

// Launches of the service that have not finished yet (from the completion words).
static int unfinished_launches(ps_service* s) {
  int n = 0;
  for (Slot& sl : s->slots) n += slot_finished(s, sl) ? 0 : 1;
  return n;
}

constexpr int kBatchDepth = 2;             // launches kept in flight before ready tasks are held back
constexpr int kBatchAhead = 6;             // a batch of kBatchSend waves may go out while fewer than this many run
constexpr unsigned long long kBatchSend = 2, kBatchMust = 16;   // batch sizes in waves of resident CTAs

}  // extern "C"

namespace {

// How many launches a set of ready blocks whose inputs are complete is sent as.  A launch
// ends with a tail in which the last CTAs finish alone; two launches on different streams
// overlap that tail with the next one's start, which one launch cannot do with itself.  So a
// large set goes out as up to kSplitMax consecutive parts of at least kSplitWaves waves of
// resident CTAs each.
constexpr unsigned long long kSplitMax = 4;
constexpr unsigned long long kSplitWavesX2 = 3;          // 1.5 waves, in halves

int parts_for(ps_service* s, const std::vector<int>& idx) {
  if (!s->opt_overlap || !s->opt_split) return 1;
  unsigned long long chunks = 0;
  for (int bi : idx) chunks += (s->blocks[bi].nelem + kChunkAuto - 1) / kChunkAuto;
  const unsigned long long per = kSplitWavesX2 * work_wave(s) / 2;
  return (int)std::max<unsigned long long>(1, std::min<unsigned long long>(kSplitMax, chunks / per));
}

// Launches `idx` (inputs complete) as `parts` consecutive launches of about equal size.
int launch_in_parts(ps_service* s, const std::vector<int>& idx, int parts) {
  unsigned long long chunks = 0;
  for (int bi : idx) chunks += (s->blocks[bi].nelem + kChunkAuto - 1) / kChunkAuto;
  std::vector<int>& part = s->part;
  size_t i = 0;
  for (int k = 0; k < parts; ++k) {
    const unsigned long long goal = chunks * (unsigned long long)(k + 1) / (unsigned long long)parts;
    part.clear();
    unsigned long long have = 0;
    for (size_t q = 0; q < i; ++q) have += (s->blocks[idx[q]].nelem + kChunkAuto - 1) / kChunkAuto;
    while (i < idx.size() && (k == parts - 1 || have < goal)) {
      have += (s->blocks[idx[i]].nelem + kChunkAuto - 1) / kChunkAuto;
      part.push_back(idx[i++]);
    }
    if (part.empty()) continue;
    int rc = build_plan(s, part, &s->plan);
    if (!rc) rc = launch_plan(s, part, s->plan, nullptr, PS_ROUND_INPUTS_COMPLETE);
    if (rc) return rc;
  }
  return PS_OK;
}

// Sends out everything the batch holds (device made current here).
int flush_batch(ps_service* s) {
  if (s->batch.empty()) return PS_OK;
  PS_CUDA(s, cudaSetDevice(s->device));
  std::vector<int> idx;
  idx.swap(s->batch);
  s->batch_chunks = 0;
  for (int bi : idx) s->blocks[bi].queued = false;
  // (a batch packed from several rounds is not split: it is sent because other launches are
  // about to finish, so its start already overlaps their tails, and more launches only add
  // their fixed cost — measured on the 12-job bursty workload: 4.56 ms split, 4.50 ms whole)
  const int parts = s->batch_rounds == 1 ? parts_for(s, idx) : 1;
  s->batch_rounds = 0;
  int rc;
  if (parts > 1) {
    rc = launch_in_parts(s, idx, parts);
  } else {
    rc = build_plan(s, idx, &s->plan);
    if (!rc) rc = launch_plan(s, idx, s->plan, nullptr, PS_ROUND_INPUTS_COMPLETE);
  }
  idx.clear();
  s->batch.swap(idx);                      // keeps the capacity
  s->batch.clear();
  return rc;
}
}  // namespace

extern "C" {

// The validated, ready blocks `idx` are to be aggregated.  Packing over time: with
// PS_OPT_OVERLAP and PS_OPT_BATCH, tasks whose inputs are complete are held back while at
// least kBatchDepth launches are still running and go out together with whatever becomes
// ready meanwhile — many small rounds then cost a few well-filled launches instead of one
// short launch each (the paper's packing of aggregation tasks, applied along time as well
// as across jobs).  An idle device gets its launch at once.  `own` (optional) is a table
// already built for exactly `idx`, used when the launch goes out alone.
static int submit_ready(ps_service* s, const std::vector<int>& idx, cudaStream_t stream, unsigned int flags,
                        Plan* own, bool own_ok, bool* own_built = nullptr) {
  const bool can_wait = s->opt_overlap && s->opt_batch && (flags & PS_ROUND_INPUTS_COMPLETE);
  if (!can_wait) {
    int rc = flush_batch(s);          // earlier rounds first: launches keep their order per block
    if (rc) return rc;
    PS_CUDA(s, cudaSetDevice(s->device));
    if (own && own_ok) return launch_plan(s, idx, *own, stream, flags);
    Plan& plan = own ? *own : s->plan;
    rc = build_plan(s, idx, &plan);
    if (rc) return rc;
    if (own && own_built) *own_built = true;
    return launch_plan(s, idx, plan, stream, flags);
  }
  const bool busy = unfinished_launches(s) >= kBatchDepth;
  if (s->batch.empty() && !busy) {         // nothing to pack with and the device has room: out it goes
    PS_CUDA(s, cudaSetDevice(s->device));
    const int parts = parts_for(s, idx);
    if (parts > 1) return launch_in_parts(s, idx, parts);
    if (own && own_ok) return launch_plan(s, idx, *own, stream, flags);
    Plan& plan = own ? *own : s->plan;
    int rc = build_plan(s, idx, &plan);
    if (rc) return rc;
    if (own && own_built) *own_built = true;
    return launch_plan(s, idx, plan, stream, flags);
  }
  s->batch_rounds++;
  for (int bi : idx) {
    Block& b = s->blocks[bi];
    b.queued = true;
    s->batch.push_back(bi);
    s->batch_chunks += (b.nelem + kChunkAuto - 1) / kChunkAuto;
  }
  // Send when the device is about to run dry; when the batch fills two waves of CTAs and
  // few launches are in flight; or when it has grown very large.  Measured on B200: with
  // everything sent at two waves a fast host puts a dozen large launches in flight, they
  // share the SMs and finish together, and the launches that depend on them start late
  // (12 packed jobs, bursty: 4.62 ms per step); holding back until the device runs dry
  // turns a step of 54 small rounds into one launch with no tail to overlap (0.21 ms);
  // this rule gives 4.44 ms and 0.18 ms.
  const unsigned long long wave = work_wave(s);
  if (!busy || (s->batch_chunks >= kBatchSend * wave && unfinished_launches(s) < kBatchAhead) ||
      s->batch_chunks >= kBatchMust * wave)
    return flush_batch(s);
  return PS_OK;
}

int ps_aggregate(ps_service* s, const ps_task* ready, int n_ready, void* stream_) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  int rc = validate_ready(s, ready, n_ready, &s->idx);
  if (rc) return rc;
  if (!has_device(s)) return PS_ERR_NO_DEVICE;
  if (s->idx.empty()) return PS_OK;
  return submit_ready(s, s->idx, static_cast<cudaStream_t>(stream_), 0u, nullptr, false);
}

static int push_batch_locked(ps_service* s, int n, const int* jobs, const int* blocks, const int* workers,
                             const void* const* ptrs);
static void unpush_locked(ps_service* s, int n, const int* jobs, const int* blocks, const int* workers);

int ps_round(ps_service* s, int n_push, const int* jobs, const int* blocks, const int* workers,
             const void* const* grad_dev_ptrs, const ps_task* ready, int n_ready, unsigned int flags, void* stream_,
             const float** params_out) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  if (flags & ~(unsigned int)PS_ROUND_INPUTS_COMPLETE) return PS_ERR_BAD_ARG;
  int rc = push_batch_locked(s, n_push, jobs, blocks, workers, grad_dev_ptrs);
  if (rc) return rc;
  rc = validate_ready(s, ready, n_ready, &s->idx);
  if (!rc && !has_device(s)) rc = PS_ERR_NO_DEVICE;
  if (!rc && !s->idx.empty()) {
    // (s->idx is scratch that a flush inside submit_ready may not touch: it only uses s->plan)
    rc = submit_ready(s, s->idx, static_cast<cudaStream_t>(stream_), flags, nullptr, false);
  }
  if (rc) {
    unpush_locked(s, n_push, jobs, blocks, workers);
    return rc;
  }
  if (params_out)
    for (size_t i = 0; i < s->idx.size(); ++i) params_out[i] = blk_p(s, s->blocks[s->idx[i]]);
  return PS_OK;
}

// Resolves a prepared round's lists against the registry as it is now.
static int resolve_prepared(ps_service* s, Prepared& r) {
  const size_t n = r.jobs.size();
  r.push_bi.resize(n);
  r.plan_ok = false;
  for (size_t i = 0; i < n; ++i) {
    const int bi = find_block(s, r.jobs[i], r.block_ids[i]);
    if (bi < 0 || !r.ptrs[i]) return PS_ERR_BAD_ARG;
    const Job& j = s->jobs[s->blocks[bi].job];
    if (r.workers[i] < 0 || r.workers[i] >= j.d.num_workers) return PS_ERR_BAD_ARG;
    if (reinterpret_cast<uintptr_t>(r.ptrs[i]) & (j.grad_esize() - 1)) return PS_ERR_ALIGN;
    r.push_bi[i] = bi;
  }
  int rc = validate_ready_ids(s, r.ready.data(), (int)r.ready.size(), &r.idx);
  if (rc) return rc;
  // self-contained: every ready block gets all of its W shards from this round's own
  // pushes and the round pushes nothing else; the table then depends on nothing but
  // the round itself (and on where the blocks live: the epoch)
  const unsigned long long gen = ++s->gen;
  std::vector<size_t> first(r.idx.size() + 1, 0);      // first[k]: offset of ready task k's worker flags
  for (size_t k = 0; k < r.idx.size(); ++k) {
    Block& b = s->blocks[r.idx[k]];
    b.mark = gen;
    b.mark_pos = (int)k;
    first[k + 1] = first[k] + (size_t)s->jobs[b.job].d.num_workers;
  }
  std::vector<unsigned char> seen(first.back(), 0);
  bool ok = true;
  size_t distinct = 0;
  for (size_t i = 0; i < n && ok; ++i) {
    const Block& b = s->blocks[r.push_bi[i]];
    if (b.mark != gen) { ok = false; break; }            // a push for a block that is not in the ready list
    unsigned char& f = seen[first[b.mark_pos] + (size_t)r.workers[i]];
    if (!f) { f = 1; ++distinct; }
  }
  ok = ok && distinct == seen.size() && n == seen.size();  // every (ready block, worker) exactly once
  r.self_contained = ok;
  r.epoch = s->epoch;
  return PS_OK;
}

int ps_round_prepare(ps_service* s, int n_push, const int* jobs, const int* blocks, const int* workers,
                     const void* const* grad_dev_ptrs, const ps_task* ready, int n_ready, unsigned int flags,
                     int* round_out) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  if (!round_out || (flags & ~(unsigned int)PS_ROUND_INPUTS_COMPLETE)) return PS_ERR_BAD_ARG;
  if (n_push < 0 || (n_push > 0 && (!jobs || !blocks || !workers || !grad_dev_ptrs))) return PS_ERR_BAD_ARG;
  if (n_ready < 0 || (n_ready > 0 && !ready)) return PS_ERR_BAD_ARG;
  Prepared r;
  r.jobs.assign(jobs, jobs + n_push);
  r.block_ids.assign(blocks, blocks + n_push);
  r.workers.assign(workers, workers + n_push);
  r.ptrs.assign(grad_dev_ptrs, grad_dev_ptrs + n_push);
  r.ready.assign(ready, ready + n_ready);
  r.flags = flags;
  int rc = resolve_prepared(s, r);
  if (rc) return rc;
  r.live = true;
  int id = -1;
  for (size_t i = 0; i < s->prepared.size(); ++i)
    if (!s->prepared[i].live) { id = (int)i; break; }
  if (id < 0) {
    s->prepared.emplace_back();
    id = (int)s->prepared.size() - 1;
  }
  s->prepared[id] = std::move(r);
  *round_out = id;
  return PS_OK;
}

int ps_round_release(ps_service* s, int round) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  if (round < 0 || round >= (int)s->prepared.size() || !s->prepared[round].live) return PS_ERR_BAD_ARG;
  s->prepared[round] = Prepared();
  return PS_OK;
}

int ps_round_run(ps_service* s, int round, void* stream_, const float** params_out) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  if (round < 0 || round >= (int)s->prepared.size() || !s->prepared[round].live) return PS_ERR_BAD_ARG;
  Prepared& r = s->prepared[round];
  if (r.epoch != s->epoch) {
    int rc = resolve_prepared(s, r);
    if (rc) return rc;
  }
  // the pushes
  const size_t n = r.push_bi.size();
  size_t done = 0;
  int rc = PS_OK;
  for (; done < n; ++done) {
    Block& b = s->blocks[r.push_bi[done]];
    const int w = r.workers[done];
    if (b.queued) {                        // its previous aggregate is still held in the batch
      rc = flush_batch(s);
      if (rc) break;
    }
    if (b.pushed[w]) { rc = PS_ERR_DUPLICATE; break; }
    if (b.nsparse > 0 && (reinterpret_cast<uintptr_t>(r.ptrs[done]) & 15u)) { rc = PS_ERR_ALIGN; break; }
    b.pushed[w] = r.ptrs[done];
    b.npushed++;
  }
  // the ready list
  if (!rc)
    for (int bi : r.idx) {
      if (s->blocks[bi].queued) {          // listed again without new pushes: not ready once its aggregate is out
        rc = flush_batch(s);
        if (rc) break;
      }
      if (s->blocks[bi].npushed != s->jobs[s->blocks[bi].job].d.num_workers) { rc = PS_ERR_NOT_READY; break; }
    }
  if (!rc && !has_device(s)) rc = PS_ERR_NO_DEVICE;
  if (!rc && !r.idx.empty()) {
    const bool reuse = r.self_contained && r.plan_ok;
    if (reuse) {
      // same blocks, same places, same pointers as last time: only the step moves on
      unsigned char* base = r.plan.bytes.data();
      PsTaskDev* tasks = reinterpret_cast<PsTaskDev*>(base + reinterpret_cast<PsTableHdr*>(base)->tasks_off);
      for (size_t i = 0; i < r.plan.order.size(); ++i) {
        const Block& b = s->blocks[r.plan.order[i]];
        set_step_fields(s->jobs[b.job], b, &tasks[i]);
      }
    }
    bool built = false;
    rc = submit_ready(s, r.idx, static_cast<cudaStream_t>(stream_), r.flags, &r.plan, reuse, &built);
    // the round's own table can be reused next time only if it was built for this round just now
    if (!reuse) r.plan_ok = !rc && r.self_contained && built;
  }
  if (rc) {
    for (size_t i = 0; i < done; ++i) {
      Block& b = s->blocks[r.push_bi[i]];
      b.pushed[r.workers[i]] = nullptr;
      b.npushed--;
    }
    return rc;
  }
  if (params_out)
    for (size_t i = 0; i < r.idx.size(); ++i) params_out[i] = blk_p(s, s->blocks[r.idx[i]]);
  return PS_OK;
}

int ps_join(ps_service* s, void* stream_) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  { int frc = flush_batch(s); if (frc) return frc; }    // held-back rounds go out first
  if (!has_device(s)) return PS_OK;
  PS_CUDA(s, cudaSetDevice(s->device));
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  // per service stream: its launches finish in order, so the latest one stands for all
  for (int w = 0; w < kWorkStreams; ++w) {
    if (s->ws_last_seq[w] == s->ws_joined_seq[w]) continue;
    s->ws_joined_seq[w] = s->ws_last_seq[w];
    Slot& sl = s->slots[s->ws_last_slot[w]];
    if (sl.seq != s->ws_last_seq[w] || slot_finished(s, sl)) continue;   // recycled (so finished) or finished
    int rc = ensure_done_event(s, sl);
    if (rc) return rc;
    PS_CUDA(s, cudaStreamWaitEvent(stream, sl.done, 0));
  }
  return PS_OK;
}

int ps_flush(ps_service* s) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  return flush_batch(s);
}

int ps_plan(ps_service* s, const ps_task* ready, int n_ready, ps_chunk_info* out, size_t cap, size_t* n_out) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  std::vector<int>& idx = s->idx;
  int rc = validate_ready(s, ready, n_ready, &idx);
  if (rc) return rc;
  Plan& plan = s->plan;
  plan.total_chunks = 0;
  if (!idx.empty()) {
    rc = build_plan(s, idx, &plan);
    if (rc) return rc;
  }
  if (n_out) *n_out = plan.total_chunks;
  if (!out || idx.empty()) return PS_OK;
  const unsigned char* base = plan.bytes.data();
  const PsTableHdr* h = reinterpret_cast<const PsTableHdr*>(base);
  const PsTaskDev* tasks = reinterpret_cast<const PsTaskDev*>(base + h->tasks_off);
  size_t k = 0;
  for (unsigned int t = 0; t < h->n_tasks && k < cap; ++t) {
    const Block& b = s->blocks[plan.order[t]];
    for (unsigned int c = 0; c < tasks[t].nchunks && k < cap; ++c, ++k) {
      ps_chunk_info& ci = out[k];
      ci.job = b.job;
      ci.block = b.id;
      ci.elem_begin = (unsigned long long)c * tasks[t].chunk_elems;
      ci.elem_count = std::min<unsigned long long>(tasks[t].chunk_elems, tasks[t].nelem - ci.elem_begin);
      ci.num_workers = s->jobs[b.job].d.num_workers;
      ci.vector_path = (int)tasks[t].vec_ok;
    }
  }
  return PS_OK;
}

int ps_pull(ps_service* s, int job, int block, const float** out) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  const int bi = find_block(s, job, block);
  if (bi < 0 || !out) return PS_ERR_BAD_ARG;
  if (!has_device(s)) return PS_ERR_NO_DEVICE;
  *out = blk_p(s, s->blocks[bi]);
  return PS_OK;
}

int ps_pull_batch(ps_service* s, const ps_task* tasks, int n, const float** out) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  if (n < 0 || (n > 0 && (!tasks || !out))) return PS_ERR_BAD_ARG;
  if (!has_device(s)) return PS_ERR_NO_DEVICE;
  for (int i = 0; i < n; ++i)
    if (find_block(s, tasks[i].job, tasks[i].block) < 0) return PS_ERR_BAD_ARG;
  for (int i = 0; i < n; ++i) out[i] = blk_p(s, s->blocks[find_block(s, tasks[i].job, tasks[i].block)]);
  return PS_OK;
}

int ps_pull_host(ps_service* s, int job, int block, float* dst, void* stream_) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  { int frc = flush_batch(s); if (frc) return frc; }    // held-back rounds go out first
  const int bi = find_block(s, job, block);
  if (bi < 0 || !dst) return PS_ERR_BAD_ARG;
  if (!has_device(s)) return PS_ERR_NO_DEVICE;
  PS_CUDA(s, cudaSetDevice(s->device));
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  Block& b = s->blocks[bi];
  ++s->call_id;
  int rc = order_after_block(s, b, stream);
  if (rc) return rc;
  PS_CUDA(s, cudaMemcpyAsync(dst, blk_p(s, b), b.nelem * sizeof(float), cudaMemcpyDeviceToHost, stream));
  return PS_OK;
}

// A copy batch that is not in use (its event exists on return).
static int free_batch(ps_service* s, int* out) {
  int batch = -1;
  for (int i = 0; i < (int)s->batches.size(); ++i)
    if (!s->batches[i].pending) { batch = i; break; }
  if (batch < 0) {
    s->batches.emplace_back();
    batch = (int)s->batches.size() - 1;
  }
  if (!s->batches[batch].ev) {
    cudaError_t e = cudaEventCreateWithFlags(&s->batches[batch].ev, cudaEventDisableTiming);
    if (e != cudaSuccess) { s->cuda_err = cudaGetErrorString(e); return PS_ERR_CUDA; }
  }
  *out = batch;
  return PS_OK;
}

// Moves the listed blocks (indices into s->blocks) to dst_ctx as ONE batch: all
// destination ranges are reserved first (nothing changes if one does not fit),
// the copies are ordered after each block's last aggregate and last move, one
// gather-copy kernel per 96 blocks (a plain cudaMemcpyAsync for a single block)
// does the transfer, and one event marks the whole batch.
static int migrate_many(ps_service* s, const std::vector<int>& bis, int dst_ctx, cudaStream_t stream) {
  struct Move { int bi; size_t noff; };
  std::vector<Move> moves;
  {
    int rc = reap_frees(s, false);
    if (rc) return rc;
  }
  for (int bi : bis) {
    Block& b = s->blocks[bi];
    if (b.ctx == dst_ctx) continue;
    size_t noff = 0;
    int rc = arena_alloc(s, dst_ctx, b.bytes, &noff, false);
    if (rc) {
      for (auto& m : moves) s->ctxs[dst_ctx].arena.release(m.noff, s->blocks[m.bi].bytes);
      return rc;
    }
    moves.push_back(Move{bi, noff});
  }
  if (moves.empty()) return PS_OK;
  auto undo = [&]() {
    for (auto& m : moves) s->ctxs[dst_ctx].arena.release(m.noff, s->blocks[m.bi].bytes);
  };
  int batch = -1;
  {
    int rc = free_batch(s, &batch);
    if (rc) { undo(); return rc; }
  }
  unsigned int waited = 0;
  for (auto& m : moves) {
    int rc = order_after_block(s, s->blocks[m.bi], stream, &waited);
    if (rc) { undo(); return rc; }
  }
  cudaError_t e = cudaSuccess;
  if (moves.size() == 1) {
    // parameters and optimizer state are one contiguous range; the step counter is host state
    Block& b = s->blocks[moves[0].bi];
    e = cudaMemcpyAsync(s->ctxs[dst_ctx].base + moves[0].noff, s->ctxs[b.ctx].base + b.off, b.bytes,
                        cudaMemcpyDeviceToDevice, stream);
  } else {
    // one launch for up to 1024 blocks (a whole model); 96 at a time where the large
    // kernel-parameter space is refused
    auto launch_some = [&](auto* args, size_t first, size_t count) {
      args->n = (int)count;
      unsigned int tiles = 0;
      for (size_t k = 0; k < count; ++k) {
        Block& b = s->blocks[moves[first + k].bi];
        args->src[k] = reinterpret_cast<const unsigned char*>(s->ctxs[b.ctx].base + b.off);
        args->dst[k] = reinterpret_cast<unsigned char*>(s->ctxs[dst_ctx].base + moves[first + k].noff);
        args->bytes[k] = b.bytes;
        args->tile_prefix[k] = tiles;
        tiles += (unsigned int)((b.bytes + kMigTile - 1) / kMigTile);
      }
      args->tile_prefix[count] = tiles;
      return (int)std::min<unsigned int>(tiles, (unsigned int)s->num_sms * 16u);
    };
    // the cost of a launch grows with its parameter bytes (measured: 21 us of host time
    // with the 28 KB table), so the smallest table that holds what is left is taken
    auto launch_as = [&](auto* args, size_t first, size_t count) {
      using A = std::remove_pointer_t<decltype(args)>;
      const int grid = launch_some(args, first, count);
      ps_migrate_kernel<A::kRanges><<<grid, 256, 0, stream>>>(*args);
      return cudaGetLastError();
    };
    size_t first = 0;
    while (first < moves.size() && e == cudaSuccess) {
      const size_t left = moves.size() - first;
      if (left > (size_t)kMigSmall && s->mig_large_ok) {
        size_t count = 0;
        if (left <= (size_t)kMigMedium) {
          static thread_local MigArgs<kMigMedium> mid;
          count = left;
          e = launch_as(&mid, first, count);
        } else {
          static thread_local MigArgs<kMigLarge> big;
          count = std::min<size_t>(kMigLarge, left);
          e = launch_as(&big, first, count);
        }
        if (e != cudaSuccess) {            // refused at launch: nothing ran; remember and take the small form
          s->mig_large_ok = false;
          e = cudaSuccess;
          continue;
        }
        first += count;
      } else {
        MigArgs<kMigSmall> small;
        const size_t count = std::min<size_t>(kMigSmall, left);
        e = launch_as(&small, first, count);
        first += count;
      }
    }
  }
  if (e == cudaSuccess) e = cudaEventRecord(s->batches[batch].ev, stream);
  if (e != cudaSuccess) { undo(); s->cuda_err = cudaGetErrorString(e); return PS_ERR_CUDA; }
  MigBatch& mb = s->batches[batch];
  mb.pending = true;
  mb.seen_call = mb.waited_call = 0;
  for (auto& m : moves) {
    Block& b = s->blocks[m.bi];
    s->pending_free.push_back(PendingFree{b.ctx, b.off, b.bytes, batch});
    b.ctx = dst_ctx;
    b.off = m.noff;
    b.mig_batch = batch;
  }
  ++s->epoch;
  return PS_OK;
}

int ps_migrate_block(ps_service* s, int job, int block, int dst_ctx, void* stream_) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  { int frc = flush_batch(s); if (frc) return frc; }    // held-back rounds go out first
  const int bi = find_block(s, job, block);
  if (bi < 0 || dst_ctx < 0 || dst_ctx >= (int)s->ctxs.size()) return PS_ERR_BAD_ARG;
  if (!has_device(s)) return PS_ERR_NO_DEVICE;
  PS_CUDA(s, cudaSetDevice(s->device));
  ++s->call_id;
  return migrate_many(s, std::vector<int>{bi}, dst_ctx, static_cast<cudaStream_t>(stream_));
}

int ps_migrate_blocks(ps_service* s, const ps_task* tasks, int n, int dst_ctx, void* stream_) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  { int frc = flush_batch(s); if (frc) return frc; }    // held-back rounds go out first
  if (n < 0 || (n > 0 && !tasks) || dst_ctx < 0 || dst_ctx >= (int)s->ctxs.size()) return PS_ERR_BAD_ARG;
  std::vector<int> bis;
  const unsigned long long gen = ++s->gen;
  for (int i = 0; i < n; ++i) {
    const int bi = find_block(s, tasks[i].job, tasks[i].block);
    if (bi < 0) return PS_ERR_BAD_ARG;
    if (s->blocks[bi].mark == gen) return PS_ERR_DUPLICATE;
    s->blocks[bi].mark = gen;
    bis.push_back(bi);
  }
  if (!has_device(s)) return PS_ERR_NO_DEVICE;
  PS_CUDA(s, cudaSetDevice(s->device));
  ++s->call_id;
  return migrate_many(s, bis, dst_ctx, static_cast<cudaStream_t>(stream_));
}

// Marks `stream`'s position as a copy batch of block b: later work on b waits for it.
static int mark_copy(ps_service* s, Block& b, cudaStream_t stream) {
  int batch = -1;
  int rc = free_batch(s, &batch);
  if (rc) return rc;
  PS_CUDA(s, cudaEventRecord(s->batches[batch].ev, stream));
  MigBatch& mb = s->batches[batch];
  mb.pending = true;
  mb.seen_call = mb.waited_call = 0;
  b.mig_batch = batch;
  return PS_OK;
}

int ps_block_export(ps_service* s, int job, int block, void* dst_dev, size_t dst_cap, size_t* bytes_out,
                    unsigned long long* step_out, void* stream_) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  { int frc = flush_batch(s); if (frc) return frc; }    // held-back rounds go out first
  const int bi = find_block(s, job, block);
  if (bi < 0) return PS_ERR_BAD_ARG;
  Block& b = s->blocks[bi];
  if (bytes_out) *bytes_out = b.bytes;
  if (step_out) *step_out = b.step;
  if (!dst_dev) return PS_OK;                       // size query
  if (dst_cap < b.bytes) return PS_ERR_BAD_ARG;
  if (!has_device(s)) return PS_ERR_NO_DEVICE;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  PS_CUDA(s, cudaSetDevice(s->device));
  ++s->call_id;
  int rc = order_after_block(s, b, stream);
  if (rc) return rc;
  PS_CUDA(s, cudaMemcpyAsync(dst_dev, s->ctxs[b.ctx].base + b.off, b.bytes, cudaMemcpyDefault, stream));
  return mark_copy(s, b, stream);
}

int ps_block_import(ps_service* s, int job, int block, const void* src_dev, size_t src_bytes,
                    unsigned long long step, void* stream_) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  { int frc = flush_batch(s); if (frc) return frc; }    // held-back rounds go out first
  const int bi = find_block(s, job, block);
  if (bi < 0 || !src_dev) return PS_ERR_BAD_ARG;
  Block& b = s->blocks[bi];
  if (src_bytes != b.bytes) return PS_ERR_BAD_ARG;
  if (!has_device(s)) return PS_ERR_NO_DEVICE;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  PS_CUDA(s, cudaSetDevice(s->device));
  ++s->call_id;
  int rc = order_after_block(s, b, stream);
  if (rc) return rc;
  PS_CUDA(s, cudaMemcpyAsync(s->ctxs[b.ctx].base + b.off, src_dev, b.bytes, cudaMemcpyDefault, stream));
  rc = mark_copy(s, b, stream);
  if (rc) return rc;
  b.step = step;
  return PS_OK;
}

int ps_unregister_block(ps_service* s, int job, int block) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  { int frc = flush_batch(s); if (frc) return frc; }    // held-back rounds go out first
  const int bi = find_block(s, job, block);
  if (bi < 0) return PS_ERR_BAD_ARG;
  Block& b = s->blocks[bi];
  if (has_device(s)) {
    PS_CUDA(s, cudaSetDevice(s->device));
    ++s->call_id;
    // everything this service enqueued for the block: its last launch, its last copy
    if (Slot* sl = pending_slot(s, b)) {
      int rc = wait_slot(s, *sl);
      if (rc) return rc;
    }
    if (b.mig_batch >= 0) {
      bool ready = false;
      int rc = batch_ready(s, b.mig_batch, true, &ready);
      if (rc) return rc;
      b.mig_batch = -1;
    }
    if (b.staging && b.staging_own) PS_CUDA(s, cudaFree(b.staging));
    b.staging = nullptr;                   // (a range of the job's region stays with the region)
  }
  s->ctxs[b.ctx].arena.release(b.off, b.bytes);
  s->jobs[b.job].block_of_id[b.id] = -1;
  b.nelem = 0;
  b.bytes = 0;
  b.npushed = 0;
  s->free_blocks.push_back(bi);
  ++s->epoch;
  return PS_OK;
}

int ps_block_stats(ps_service* s, int job, int block, double* sq_out, unsigned long long* step_out) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  { int frc = flush_batch(s); if (frc) return frc; }    // held-back rounds go out first
  const int bi = find_block(s, job, block);
  if (bi < 0) return PS_ERR_BAD_ARG;
  Block& b = s->blocks[bi];
  if (step_out) *step_out = b.step;
  if (!sq_out) return PS_OK;
  *sq_out = 0.0;
  if (!has_device(s) || b.last_slot < 0) return PS_OK;
  PS_CUDA(s, cudaSetDevice(s->device));
  if (Slot* sl = pending_slot(s, b)) {
    int rc = wait_slot(s, *sl);
    if (rc) return rc;
  }
  PsStat st;
  PS_CUDA(s, cudaMemcpy(&st, s->stats_dev + b.stat_idx, sizeof st, cudaMemcpyDeviceToHost));
  *sq_out = st.sqnorm;
  return PS_OK;
}

// Waits for the block's last aggregate and reads its statistics record.
static int read_stat(ps_service* s, Block& b, PsStat* st) {
  std::memset(st, 0, sizeof *st);
  if (!has_device(s) || b.last_slot < 0) return PS_OK;
  PS_CUDA(s, cudaSetDevice(s->device));
  if (Slot* sl = pending_slot(s, b)) {
    int rc = wait_slot(s, *sl);
    if (rc) return rc;
  }
  PS_CUDA(s, cudaMemcpy(st, s->stats_dev + b.stat_idx, sizeof *st, cudaMemcpyDeviceToHost));
  return PS_OK;
}

int ps_block_profile(ps_service* s, int job, int block, double* busy_us_out, double* span_us_out) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  { int frc = flush_batch(s); if (frc) return frc; }    // held-back rounds go out first
  const int bi = find_block(s, job, block);
  if (bi < 0) return PS_ERR_BAD_ARG;
  PsStat st;
  int rc = read_stat(s, s->blocks[bi], &st);
  if (rc) return rc;
  if (busy_us_out) *busy_us_out = st.busy_ns * 1e-3;
  if (span_us_out) *span_us_out = st.t_last > st.t_first ? (st.t_last - st.t_first) * 1e-3 : 0.0;
  return PS_OK;
}

int ps_job_profile(ps_service* s, int job, double* busy_us_out, double* span_us_out, int* blocks_out) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  { int frc = flush_batch(s); if (frc) return frc; }    // held-back rounds go out first
  if (job < 0 || job >= (int)s->jobs.size()) return PS_ERR_BAD_ARG;
  double busy = 0.0;
  unsigned long long first = ~0ull, last = 0;
  int n = 0;
  for (int bi : s->jobs[job].block_of_id) {
    if (bi < 0) continue;
    PsStat st;
    int rc = read_stat(s, s->blocks[bi], &st);
    if (rc) return rc;
    if (st.t_last == 0) continue;          // never profiled
    busy += st.busy_ns * 1e-3;
    first = std::min(first, st.t_first);
    last = std::max(last, st.t_last);
    ++n;
  }
  if (busy_us_out) *busy_us_out = busy;
  if (span_us_out) *span_us_out = n && last > first ? (last - first) * 1e-3 : 0.0;
  if (blocks_out) *blocks_out = n;
  return PS_OK;
}

int ps_block_state(ps_service* s, int job, int block, const float** s0, const float** s1, int* ctx_out) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  const int bi = find_block(s, job, block);
  if (bi < 0) return PS_ERR_BAD_ARG;
  Block& b = s->blocks[bi];
  if (ctx_out) *ctx_out = b.ctx;
  if (s0) *s0 = has_device(s) ? blk_s0(s, b) : nullptr;
  if (s1) *s1 = has_device(s) ? blk_s1(s, b) : nullptr;
  return PS_OK;
}

int ps_set_option(ps_service* s, int option, long long value) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  { int frc = flush_batch(s); if (frc) return frc; }    // held-back rounds go out first
  ++s->epoch;                              // chunking, sorting, kernel choice: prepared tables are rebuilt
  switch (option) {
    case PS_OPT_CHUNK_ELEMS:
      if (value < 0 || value > (long long)kMaxChunk || (value % 1024) != 0) return PS_ERR_BAD_ARG;
      s->opt_chunk = value;
      return PS_OK;
    case PS_OPT_CTAS_PER_SM:
      if (value < 0 || value > 32) return PS_ERR_BAD_ARG;
      s->opt_ctas = value;
      return PS_OK;
    case PS_OPT_SORT_TASKS:
      s->opt_sort = value ? 1 : 0;
      return PS_OK;
    case PS_OPT_KERNEL:
      if (value < 0 || value > 2) return PS_ERR_BAD_ARG;
      s->opt_kernel = value;
      return PS_OK;
    case PS_OPT_PROFILE:
      s->opt_profile = value ? 1 : 0;
      return PS_OK;
    case PS_OPT_OVERLAP:
      s->opt_overlap = value ? 1 : 0;
      return PS_OK;
    case PS_OPT_INLINE_TABLE:
      s->opt_inline = value ? 1 : 0;
      return PS_OK;
    case PS_OPT_PDL:
      s->opt_pdl = value ? 1 : 0;
      return PS_OK;
    case PS_OPT_BATCH:
      s->opt_batch = value ? 1 : 0;
      return PS_OK;
    case PS_OPT_SPLIT:
      s->opt_split = value ? 1 : 0;
      return PS_OK;
    case PS_OPT_WAIT_CYCLES:
      if (value < 1) return PS_ERR_BAD_ARG;
      s->opt_wait_cycles = value;
      return PS_OK;
    case PS_OPT_WORK_STREAMS:
      if (value < 1 || value > kWorkStreams) return PS_ERR_BAD_ARG;
      s->opt_streams = value;
      s->next_work = 0;
      return PS_OK;
    default:
      return PS_ERR_BAD_ARG;
  }
}

int ps_get_option(ps_service* s, int option, long long* out) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  if (!out) return PS_ERR_BAD_ARG;
  switch (option) {
    case PS_OPT_CHUNK_ELEMS: *out = s->opt_chunk; return PS_OK;
    case PS_OPT_CTAS_PER_SM: *out = s->opt_ctas; return PS_OK;
    case PS_OPT_SORT_TASKS: *out = s->opt_sort; return PS_OK;
    case PS_OPT_KERNEL: *out = s->opt_kernel; return PS_OK;
    case PS_OPT_PROFILE: *out = s->opt_profile; return PS_OK;
    case PS_OPT_OVERLAP: *out = s->opt_overlap; return PS_OK;
    case PS_OPT_INLINE_TABLE: *out = s->opt_inline; return PS_OK;
    case PS_OPT_PDL: *out = s->opt_pdl; return PS_OK;
    case PS_OPT_WORK_STREAMS: *out = s->opt_streams; return PS_OK;
    case PS_OPT_BATCH: *out = s->opt_batch; return PS_OK;
    case PS_OPT_WAIT_CYCLES: *out = s->opt_wait_cycles; return PS_OK;
    case PS_OPT_SPLIT: *out = s->opt_split; return PS_OK;
    default: return PS_ERR_BAD_ARG;
  }
}

int ps_arena_info(ps_service* s, int ctx, size_t* used_out, size_t* largest_free_out) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  if (ctx < 0 || ctx >= (int)s->ctxs.size()) return PS_ERR_BAD_ARG;
  if (has_device(s)) {
    int rc = reap_frees(s, false);
    if (rc) return rc;
  }
  if (used_out) *used_out = s->ctxs[ctx].arena.used();
  if (largest_free_out) *largest_free_out = s->ctxs[ctx].arena.largest_free();
  return PS_OK;
}

int ps_registry_info(ps_service* s, size_t* jobs_out, size_t* blocks_out, size_t* block_entries_out) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  if (jobs_out) *jobs_out = s->jobs.size();
  if (blocks_out) *blocks_out = s->blocks.size() - s->free_blocks.size();
  if (block_entries_out) *block_entries_out = s->blocks.size();
  return PS_OK;
}

int ps_arena_export(ps_service* s, int ctx, unsigned char* handle_out, size_t* bytes_out) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  if (ctx < 0 || ctx >= (int)s->ctxs.size() || !handle_out) return PS_ERR_BAD_ARG;
  if (!has_device(s)) return PS_ERR_NO_DEVICE;
  PS_CUDA(s, cudaSetDevice(s->device));
  cudaIpcMemHandle_t h;
  static_assert(sizeof(h) == PS_PEER_HANDLE_BYTES, "handle size");
  PS_CUDA(s, cudaIpcGetMemHandle(&h, s->ctxs[ctx].base));
  std::memcpy(handle_out, &h, sizeof(h));
  if (bytes_out) *bytes_out = s->ctxs[ctx].arena.capacity();
  return PS_OK;
}

int ps_block_location(ps_service* s, int job, int block, int* ctx_out, size_t* offset_out, size_t* section_out) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  const int bi = find_block(s, job, block);
  if (bi < 0) return PS_ERR_BAD_ARG;
  const Block& b = s->blocks[bi];
  if (ctx_out) *ctx_out = b.ctx;
  if (offset_out) *offset_out = b.off;
  if (section_out) *section_out = b.sec;
  return PS_OK;
}

int ps_launch_info(ps_service* s, unsigned long long* launches, int* grid, int* block, const char** name) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  { int frc = flush_batch(s); if (frc) return frc; }    // held-back rounds go out first
  if (launches) *launches = s->launches;
  if (grid) *grid = s->last_grid;
  if (block) *block = s->last_block;
  if (name) *name = s->last_kernel;
  return PS_OK;
}

int ps_launch_stats(ps_service* s, int variant, unsigned long long* launches_out, unsigned long long* bytes_out,
                    const char** name_out) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  { int frc = flush_batch(s); if (frc) return frc; }    // held-back rounds go out first
  if (variant < 0 || variant >= kVariants) return PS_ERR_BAD_ARG;
  static const char* const names[kVariants] = {"ps_aggregate_ldg_kernel", "ps_aggregate_inline_kernel",
                                               "ps_aggregate_bulk_kernel"};
  if (launches_out) *launches_out = s->var_launches[variant];
  if (bytes_out) *bytes_out = s->var_bytes[variant];
  if (name_out) *name_out = names[variant];
  return PS_OK;
}

int ps_device_status(ps_service* s, int* status_out) {
  if (!alive(s)) return PS_ERR_BAD_HANDLE;
  std::lock_guard<std::mutex> lk(s->mu);
  { int frc = flush_batch(s); if (frc) return frc; }    // held-back rounds go out first
  if (!status_out) return PS_ERR_BAD_ARG;
  *status_out = 0;
  if (!has_device(s)) return PS_OK;
  PS_CUDA(s, cudaSetDevice(s->device));
  PS_CUDA(s, cudaDeviceSynchronize());
  PS_CUDA(s, cudaMemcpy(status_out, s->status_dev, sizeof(int), cudaMemcpyDeviceToHost));
  return PS_OK;
}

const char* ps_strerror(int status) {
  switch (status) {
    case PS_OK: return "ok";
    case PS_ERR_BAD_HANDLE: return "bad service handle";
    case PS_ERR_BAD_ARG: return "bad argument";
    case PS_ERR_DUPLICATE: return "duplicate block, push or task";
    case PS_ERR_NOT_READY: return "a listed task has fewer than W pushes";
    case PS_ERR_ALIGN: return "gradient pointer not aligned to its element size";
    case PS_ERR_NOMEM: return "out of arena, device or host memory";
    case PS_ERR_CUDA: return "CUDA runtime error";
    case PS_ERR_NO_DEVICE: return "service has no device (planning only)";
    case PS_ERR_TOO_LARGE: return "block larger than PS_NOALLOC_MAX_ELEMS";
    default: return "unknown status";
  }
}

const char* ps_last_cuda_error(ps_service* s) { return alive(s) ? s->cuda_err.c_str() : ""; }

const char* ps_version(void) { return "ps_b200 0.1 (sm_100a)"; }

}  // extern "C"

// ---------------------------------------------------------------------------
// ps_aggregate_block_noalloc: one block, no allocation of any kind.
//
// The aggregation kernel needs a little global memory besides its inputs and
// outputs: the task table it walks, the work counter, one partial sum per chunk
// and the statistics record.  Here that scratch is a fixed array in the
// library's device image.  In host code the array's name is only a handle for
// the runtime, not a device address: the address comes from
// cudaGetSymbolAddress, once per device with that device current, and is what
// the kernels are given.  Device code (the two small kernels below) names the
// array directly.
// ---------------------------------------------------------------------------
namespace psb {

constexpr unsigned int kNaChunk = 8192;                                   // elements per chunk
constexpr size_t kNaMaxChunks = PS_NOALLOC_MAX_ELEMS / kNaChunk;          // 2048
constexpr size_t kNaTaskOff = sizeof(PsTableHdr);                         // 48
constexpr size_t kNaStartsOff = kNaTaskOff + sizeof(PsTaskDev);           // 176
constexpr size_t kNaPtrsOff = 192;
constexpr size_t kNaJobOff = kNaPtrsOff + PS_MAX_WORKERS * sizeof(void*); // 2240
constexpr size_t kNaStatOff = kNaJobOff + sizeof(PsJobDev);               // 2304
constexpr size_t kNaPartOff = 2560;
constexpr size_t kNaScratchBytes = kNaPartOff + kNaMaxChunks * sizeof(double);   // 18688
static_assert(kNaStartsOff + sizeof(unsigned int) <= kNaPtrsOff, "scratch layout");
static_assert(kNaStatOff + sizeof(PsStat) <= kNaPartOff, "scratch layout");
static_assert(kNaScratchBytes <= 20480, "scratch stays at 20 KB");

static __device__ __align__(256) unsigned char g_noalloc_scratch[20480];

struct NoAllocArgs {            // passed by value as kernel parameters (< 4 KB)
  PsJobDev job;
  PsTaskDev task;
  const void* shards[PS_MAX_WORKERS];
};

// Writes this call's task table into the scratch array; everything that must
// start at zero (work counter, ticket, statistics) is rewritten on every call
// because the array keeps the previous call's contents.
__global__ void ps_noalloc_setup_kernel(NoAllocArgs a) {
  unsigned char* base = g_noalloc_scratch;
  const unsigned int t = threadIdx.x;
  if (t < (unsigned int)a.job.W) reinterpret_cast<const void**>(base + kNaPtrsOff)[t] = a.shards[t];
  if (t == 0) {
    PsTableHdr h;
    h.counter = 0;
    h.n_tasks = 1;
    h.total_chunks = a.task.nchunks;
    h.chunk_elems = kNaChunk;
    h.tasks_off = (unsigned int)kNaTaskOff;
    h.starts_off = (unsigned int)kNaStartsOff;
    h.ptrs_off = (unsigned int)kNaPtrsOff;
    h.parts_per_chunk = 1;
    h.profile = 0;
    h.sparse_off = 0;
    h.exited = 0;
    h.wait_units = 0;
    *reinterpret_cast<PsTableHdr*>(base) = h;
    *reinterpret_cast<PsTaskDev*>(base + kNaTaskOff) = a.task;     // ticket = 0 inside
    *reinterpret_cast<unsigned int*>(base + kNaStartsOff) = 0;
    *reinterpret_cast<PsJobDev*>(base + kNaJobOff) = a.job;
    PsStat z;
    z.sqnorm = 0.0;
    z.step = 0;
    z.busy_ns = z.t_first = z.t_last = z._r0 = 0;
    *reinterpret_cast<PsStat*>(base + kNaStatOff) = z;
  }
}

__global__ void ps_noalloc_finish_kernel(double* out) {
  *out = reinterpret_cast<const PsStat*>(g_noalloc_scratch + kNaStatOff)->sqnorm;
}

struct NoAllocDevice {
  unsigned char* scratch = nullptr;   // device address of g_noalloc_scratch on this device
  int num_sms = 0;
};
constexpr int kNaMaxDevices = 64;
static NoAllocDevice g_na_dev[kNaMaxDevices];
static std::mutex g_na_mu;

}  // namespace psb

extern "C" int ps_aggregate_block_noalloc(const ps_job_desc* job, unsigned long long step, size_t nelem,
                                          float* params, float* state0, float* state1,
                                          const void* const* shard_ptrs, double* sqnorm_out, void* stream_) {
  if (!job || !params || !state0 || !shard_ptrs || step < 1 || nelem == 0) return PS_ERR_BAD_ARG;
  if (job->opt != PS_SGD && job->opt != PS_ADAM) return PS_ERR_BAD_ARG;
  if (job->grad_dtype != PS_F32 && job->grad_dtype != PS_BF16) return PS_ERR_BAD_ARG;
  if (job->num_workers < 1 || job->num_workers > PS_MAX_WORKERS) return PS_ERR_BAD_ARG;
  if (job->opt == PS_ADAM && !state1) return PS_ERR_BAD_ARG;
  if (nelem > PS_NOALLOC_MAX_ELEMS) return PS_ERR_TOO_LARGE;
  const uintptr_t esz = job->grad_dtype == PS_BF16 ? 2 : 4;
  // `all` decides between 128-bit and scalar accesses: parameters, state and shards only
  // (the norm is one double written by a single thread and needs 8-byte alignment, no more)
  uintptr_t all = reinterpret_cast<uintptr_t>(params) | reinterpret_cast<uintptr_t>(state0) |
                  reinterpret_cast<uintptr_t>(state1);
  if ((all & 3u) || (reinterpret_cast<uintptr_t>(sqnorm_out) & 7u)) return PS_ERR_ALIGN;
  for (int w = 0; w < job->num_workers; ++w) {
    if (!shard_ptrs[w]) return PS_ERR_BAD_ARG;
    if (reinterpret_cast<uintptr_t>(shard_ptrs[w]) & (esz - 1)) return PS_ERR_ALIGN;
    all |= reinterpret_cast<uintptr_t>(shard_ptrs[w]);
  }

  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kNaMaxDevices) return PS_ERR_CUDA;
  NoAllocDevice nd;
  {
    // first call on this device: look the scratch array's address up (the
    // device is current, as the runtime requires) and remember it
    std::lock_guard<std::mutex> lk(g_na_mu);
    if (!g_na_dev[dev].scratch) {
      void* ptr = nullptr;
      if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) return PS_ERR_CUDA;
      int sms = 0;
      if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
        return PS_ERR_CUDA;
      g_na_dev[dev].num_sms = sms;
      g_na_dev[dev].scratch = static_cast<unsigned char*>(ptr);
    }
    nd = g_na_dev[dev];
  }

  NoAllocArgs a;
  std::memset(&a, 0, sizeof a);
  a.job.opt = job->opt; a.job.grad_dtype = job->grad_dtype; a.job.W = job->num_workers;
  a.job.lr = job->lr; a.job.mom = job->momentum; a.job.wd = job->weight_decay;
  a.job.b1 = job->beta1; a.job.b2 = job->beta2;
  a.job.omb1 = 1.0f - job->beta1;
  a.job.omb2 = 1.0f - job->beta2;
  a.job.eps = job->eps; a.job.gs = job->grad_scale;
  a.task.p = params; a.task.s0 = state0; a.task.s1 = state1;
  a.task.nelem = nelem;
  a.task.shard_row = 0;
  a.task.first_chunk = 0;
  a.task.nchunks = (unsigned int)((nelem + kNaChunk - 1) / kNaChunk);
  a.task.ticket = 0;
  a.task.ss_t = (float)((double)job->lr / (1.0 - std::pow((double)job->beta1, (double)step)));
  a.task.sbc2_t = (float)std::sqrt(1.0 - std::pow((double)job->beta2, (double)step));
  a.task.job = 0;
  a.task.stat_idx = 0;
  a.task.step = step;
  a.task.vec_ok = (all & 15u) ? 0u : 1u;
  a.task.tile_elems = 0;
  a.task.chunk_elems = kNaChunk;
  for (int w = 0; w < job->num_workers; ++w) a.shards[w] = shard_ptrs[w];

  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  unsigned char* sc = nd.scratch;
  cudaGetLastError();   // an error left behind by unrelated earlier work is not this call's
  ps_noalloc_setup_kernel<<<1, PS_MAX_WORKERS, 0, stream>>>(a);
  const int grid = (int)std::min<unsigned long long>(a.task.nchunks, (unsigned long long)nd.num_sms * 3ull);
  ps_aggregate_ldg_kernel<<<grid, kThreads, 0, stream>>>(sc, reinterpret_cast<const PsJobDev*>(sc + kNaJobOff),
                                                         reinterpret_cast<PsStat*>(sc + kNaStatOff),
                                                         reinterpret_cast<double*>(sc + kNaPartOff), nullptr, 0ull);
  if (sqnorm_out) ps_noalloc_finish_kernel<<<1, 1, 0, stream>>>(sqnorm_out);
  return cudaGetLastError() == cudaSuccess ? PS_OK : PS_ERR_CUDA;
}
