/* ps_b200.h — C ABI of the packed model-aggregation service for one B200.
 *
 * The service stands for the Aggregator of Parameter Service: it holds the
 * master copy of every registered tensor block, receives the W workers'
 * gradient shards (Push), sums them, applies the job's optimizer to the
 * master copy in the same pass and exposes the result (Pull).  Blocks of many
 * jobs are packed into one kernel launch.  Requests are keyed by
 * (job ID, block ID) as in the paper's Appendix A.
 *
 * Conventions
 *  - Every function returns PS_OK (0) or a negative ps_status; nothing throws
 *    or aborts across this boundary.  On error the service is unchanged unless
 *    the function's comment says otherwise.
 *  - "device pointer" = address in the memory of the service's GPU.
 *    "host pointer"   = ordinary process memory (pinned or pageable).
 *  - `stream` arguments are a cudaStream_t passed as void* (NULL = the legacy
 *    default stream).  Work is enqueued; functions return without waiting
 *    unless stated.
 *  - The service owns parameters and optimizer state; the caller owns every
 *    gradient buffer.  The library never frees caller memory.
 *  - A service is used from one host thread at a time (calls are serialised by
 *    an internal mutex).
 *
 * Arithmetic (the paper's Section 2 says only that the server updates the
 * master copy using the aggregated result; the optimizer equations are this
 * library's reading).  For block b of job j at its t-th aggregate, element i:
 *     G  = g_0[i] + g_1[i] + ... + g_{W-1}[i]      binary32, this order
 *     G  = G * grad_scale
 *     d  = G + wd * p[i]
 *     SGD : v' = mom * v[i] + d;            p' = p[i] - lr * v'
 *     ADAM: m' = b1*m[i] + (1-b1)*d;  v' = b2*v[i] + (1-b2)*d*d
 *           p' = p[i] - (lr/(1-b1^t)) * m' / (sqrt(v')/sqrt(1-b2^t) + eps)
 * Every operation is one IEEE-754 binary32 round-to-nearest operation with no
 * fused multiply-add; bf16 gradients are widened exactly.  The per-block
 * statistic is sum_i G*G in binary64.
 */
#ifndef PS_B200_H
#define PS_B200_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ps_service ps_service; /* opaque */

typedef enum { PS_SGD = 0, PS_ADAM = 1 } ps_opt;
typedef enum { PS_F32 = 0, PS_BF16 = 1 } ps_dtype; /* gradient type; parameters and state are fp32 */

typedef enum {
  PS_OK = 0,
  PS_ERR_BAD_HANDLE = -1, /* NULL or destroyed service */
  PS_ERR_BAD_ARG = -2,    /* unknown job/block/worker/context, W < 1, nelem = 0, NULL pointer, ... */
  PS_ERR_DUPLICATE = -3,  /* block registered twice; worker pushed twice; task listed twice */
  PS_ERR_NOT_READY = -4,  /* a listed task has fewer than W pushes: whole call rejected */
  PS_ERR_ALIGN = -5,      /* gradient pointer not aligned to its element size */
  PS_ERR_NOMEM = -6,      /* context arena (or host/device allocation) exhausted */
  PS_ERR_CUDA = -7,       /* a CUDA runtime call failed; see ps_last_cuda_error */
  PS_ERR_NO_DEVICE = -8,  /* service was created without a device (planning only) */
  PS_ERR_TOO_LARGE = -9   /* ps_aggregate_block_noalloc: nelem above PS_NOALLOC_MAX_ELEMS */
} ps_status;

typedef struct {
  int opt;          /* ps_opt */
  int grad_dtype;   /* ps_dtype */
  int num_workers;  /* W, 1..PS_MAX_WORKERS */
  float lr, momentum, weight_decay, beta1, beta2, eps, grad_scale;
} ps_job_desc;

typedef struct { int job, block; } ps_task;

#define PS_MAX_WORKERS 256
#define PS_DEVICE_NONE (-1)

/* Options for ps_set_option / ps_get_option. */
enum {
  PS_OPT_CHUNK_ELEMS = 1,  /* elements per (job,block,chunk) descriptor; 0 = automatic (8192).
                              Must be a multiple of 1024 (<= 2^20) when non-zero. */
  PS_OPT_CTAS_PER_SM = 2,  /* persistent CTAs per SM; 0 = automatic */
  PS_OPT_SORT_TASKS = 3,   /* 1 (default): heaviest chunks first inside a launch; 0: caller's order */
  PS_OPT_OVERLAP = 6,      /* 1: ps_aggregate runs its launch on service-owned streams, ordered after
                              the work enqueued on `stream` at call time and after earlier launches
                              that touch the same blocks, but NOT joined back into `stream`:
                              consecutive launches overlap (the tail of one with the head of the
                              next).  The caller joins with ps_join(svc, stream) before it reuses
                              gradient buffers or reads results on its own streams; ps_pull_host,
                              ps_block_stats, ps_block_profile, ps_migrate_block and ps_push_host
                              order themselves after the block's last launch in either mode.
                              A small launch that must follow an unfinished one (a block aggregated
                              again) goes to that launch's stream, where stream order is the
                              dependency; large launches rotate over the service's streams and wait
                              for exactly the launches they depend on.  What only the host has to
                              know (may a table slot be reused, has a block's last launch finished,
                              how many launches are running) it reads from a word that the last CTA
                              of every launch stores to page-locked host memory.
                              Default 0: every launch is enqueued on `stream` itself. */
  PS_OPT_INLINE_TABLE = 7, /* 1 (default): a launch whose task table fits 3968 bytes (a round of a few
                              tensors) and has few chunks passes the table as a kernel parameter, one
                              CTA per chunk: no upload.  0: always upload the table.  Same results. */
  PS_OPT_PDL = 8,          /* 1 (default): such small launches carry the programmatic-stream-serialization
                              launch attribute: the kernel's prologue (task lookup in its parameters)
                              overlaps the tail of the previous launch of the same stream, and the
                              kernel waits for that launch to complete before it touches any data.
                              0: plain launches.  Same results. */
  PS_OPT_BATCH = 10,       /* 1 (default), effective with PS_OPT_OVERLAP for rounds given with
                              PS_ROUND_INPUTS_COMPLETE: packing over time.  While at least two launches
                              of the service are still running, such a round is not launched but held
                              back and packed into ONE launch with the rounds that follow it; the batch
                              goes out when the device is about to run dry, when it fills two waves of
                              CTAs while fewer than six launches are running, when it fills sixteen
                              waves, at ps_join / ps_flush, and before any call that reads or moves the
                              blocks' state (ps_block_stats, ps_pull_host, ps_migrate_block, a push for a
                              block that waits in the batch, ...).  An idle device gets every round at
                              once.  Results are identical; what changes is how many launches carry
                              them.  0: one launch per round. */
  PS_OPT_SPLIT = 12,       /* 1 (default), with PS_OPT_OVERLAP and PS_OPT_BATCH for rounds given with
                              PS_ROUND_INPUTS_COMPLETE: a set of ready blocks that fills several waves
                              of CTAs is sent as up to four consecutive launches of at least a wave and
                              a half each, on different streams, so that the tail of one overlaps the
                              start of the next.  Only a single round is cut this way; what was packed
                              from several rounds goes out as one launch.  0: one launch.  Same results. */
  PS_OPT_WAIT_CYCLES = 11, /* bulk-copy kernel: how many SM clock cycles a warp waits for a ring stage
                              before it gives up, records the failure in the status word
                              (ps_device_status) and lets the launch end; default 4e9 (about 2 s).
                              Results of a launch that gave up are undefined. */
  PS_OPT_WORK_STREAMS = 9, /* with PS_OPT_OVERLAP: launches rotate over this many service-owned streams
                              (1..8, default 4) */
  PS_OPT_PROFILE = 5,      /* 1: aggregates record per-task device time (see ps_block_profile);
                              costs a few atomics per chunk; direct-load kernel only; default 0 */
  PS_OPT_KERNEL = 4        /* kernel variant: 0 = automatic (direct loads), 1 = direct loads,
                              2 = bulk-copy ring (shards staged through shared memory by the TMA
                              unit); results are identical except for the rounding of the
                              per-block norm */
};

/* Creates an Aggregator service on GPU `device` with `num_contexts` contexts
 * (paper Section 3.1: an Aggregator holds the master copies of the tensors
 * assigned to it; here a context is one arena of `arena_bytes_per_ctx` bytes of
 * device memory that holds parameters and optimizer state).  Allocates the
 * arenas with cudaMalloc.  device = PS_DEVICE_NONE builds a planning-only
 * service: registration, push bookkeeping and ps_plan work, no device memory
 * exists and ps_aggregate/ps_pull/ps_migrate_block return PS_ERR_NO_DEVICE.
 * Errors: BAD_ARG (out NULL, num_contexts < 1), NOMEM, CUDA. */
int ps_create(ps_service** out, int device, int num_contexts, size_t arena_bytes_per_ctx);

/* Frees the arenas and all service-owned memory after synchronising the
 * device work the service enqueued.  Pointers from ps_pull become invalid. */
int ps_destroy(ps_service* svc);

/* Registers a training job (paper Section 4: Agents register the job with the
 * manager; Appendix A: the job ID travels with every request).  `desc` is a
 * host pointer, copied.  *job_out receives the job ID (0, 1, 2, ...).
 * Errors: BAD_ARG (opt/dtype unknown, W out of range, NULL). */
int ps_register_job(ps_service* svc, const ps_job_desc* desc, int* job_out);

/* Registers block `block` (>= 0, caller-chosen, unique within the job) of
 * `nelem` fp32 parameters in context `ctx` — the per-tensor Init of the
 * paper's Appendix A.  `init_params_or_null` may be a host or a device pointer
 * to nelem floats (copied before return) or NULL (zeros).  Optimizer state
 * starts at zero and the step counter at 0.  Synchronous.
 * Errors: BAD_ARG, DUPLICATE, NOMEM, CUDA. */
int ps_register_block(ps_service* svc, int job, int block, size_t nelem, int ctx,
                      const float* init_params_or_null);

/* Push (paper Section 4, Appendix A): records worker `worker`'s gradient shard
 * for (job, block).  Zero-copy: `grad_dev_ptr` is a device pointer to nelem
 * contiguous values of the job's grad_dtype; it must stay valid and unmodified
 * until the ps_aggregate that consumes it has completed on its stream.  The
 * task is ready once all W workers have pushed.  16-byte aligned pointers take
 * the vector path, others a scalar path with identical results.  Any address
 * the service's GPU can load from will do: its own memory, a mapped peer buffer
 * (ps_peer_open), or page-locked host memory (cudaHostAlloc / cudaHostRegister
 * under unified addressing), which the kernel then reads over PCIe in place.
 * Errors: BAD_ARG, DUPLICATE (this worker already pushed this iteration; the
 * paper has one request per task per iteration), ALIGN. */
int ps_push(ps_service* svc, int job, int block, int worker, const void* grad_dev_ptr);

/* Row-sparse Push for embedding-like blocks (no counterpart in the paper, which
 * never mentions sparsity; the result is defined as the DENSE one): the worker
 * sends only the rows of the block it touched — `row_ids` = n_rows block-local
 * row indices, strictly increasing (device int32 array, caller's contract, not
 * checked), `values` = those rows packed back to back, row_len elements each, of
 * the job's grad_dtype (device).  Rows that are not listed count as +0.0, so
 * parameters and state come out bit-identical to pushing the dense shard with
 * zero rows, and momentum decay / weight decay still reach every row; only the
 * rows that exist are read.  Requirements: nelem a multiple of row_len;
 * row_len * element size a multiple of 16 bytes; `values` 16-byte aligned (else
 * PS_ERR_ALIGN); W <= 32.  n_rows may be 0 (both pointers still non-NULL).  A
 * block may receive dense pushes from some workers and row-sparse ones from
 * others, all with the same row_len within an iteration; the dense shards of
 * such a block are streamed row by row with 128-bit loads as well, so they must
 * be 16-byte aligned too: whichever push comes second (the row-sparse one after
 * an unaligned dense one, or the unaligned dense one after a row-sparse one) is
 * rejected with PS_ERR_ALIGN.  Launches that carry such tasks always use the
 * direct-load kernel.
 * Errors: BAD_ARG, ALIGN, DUPLICATE. */
int ps_push_rows(ps_service* svc, int job, int block, int worker, const int* row_ids_dev, int n_rows,
                 int row_len, const void* values_dev);

/* n row-sparse pushes in one call (host arrays of length n).  All-or-nothing. */
int ps_push_rows_batch(ps_service* svc, int n, const int* jobs, const int* blocks, const int* workers,
                       const int* const* row_ids_dev, const int* n_rows, const int* row_lens,
                       const void* const* values_dev);

/* n pushes in one call (host arrays of length n).  All-or-nothing. */
int ps_push_batch(ps_service* svc, int n, const int* jobs, const int* blocks, const int* workers,
                  const void* const* grad_dev_ptrs);

/* Push from host memory: copies nelem gradient values from `grad_host_ptr`
 * into a service-owned device staging buffer (allocated at the job's first push
 * from host memory, see ps_push_host_batch) with cudaMemcpyAsync on `stream`,
 * then records the push.  The host
 * buffer must stay valid until that copy completes; the ps_aggregate that
 * consumes the push must be enqueued on the same stream (or one ordered after
 * it).  Errors as ps_push, plus NOMEM, CUDA, NO_DEVICE. */
int ps_push_host(ps_service* svc, int job, int block, int worker, const void* grad_host_ptr,
                 void* stream);

/* n pushes from host memory in one call (host arrays of length n), all-or-nothing.
 * The staging buffers of a job's blocks are ONE device region, laid out block after
 * block in id order, each block W rows of round_up(nelem * element size, 256) bytes
 * (allocated at the job's first push from host memory, for the blocks it has then).
 * Shards that lie in the caller's host buffer in that same layout — block after
 * block, worker after worker, rows padded to 256 bytes — are neighbours on both
 * sides and are sent as ONE copy, padding included: a round of many small tensors
 * then costs a few large copies instead of one small copy per (block, worker).
 * Any other host layout works too, with one copy per shard.  The host buffers must
 * stay valid until the copies complete; the ps_aggregate that consumes the pushes
 * is enqueued on the same stream (or one ordered after it).
 * Errors: those of ps_push_host; DUPLICATE also for a (block, worker) listed twice. */
int ps_push_host_batch(ps_service* svc, int n, const int* jobs, const int* blocks, const int* workers,
                       const void* const* grad_host_ptrs, void* stream);

/* Aggregates every task in `ready` (host array, any mix of jobs) in ONE kernel
 * launch on `stream`: sum of the W shards in worker order, optimizer update of
 * the master copy and state, per-block squared gradient norm (the paper's
 * Section 3.3 packs many jobs' aggregation tasks onto a shared Aggregator;
 * Figure 1: update after all workers pushed).  On success each listed block's
 * pushes are consumed and its step counter is incremented.  n_ready = 0 is a
 * no-op.  If a listed block is under migration the launch is ordered after the
 * copy (Appendix B, "Data Consistency").
 * Errors (nothing launched, nothing changed): BAD_ARG, DUPLICATE, NOT_READY,
 * NO_DEVICE, NOMEM, CUDA. */
int ps_aggregate(ps_service* svc, const ps_task* ready, int n_ready, void* stream);

/* Makes `stream` wait for every ps_aggregate launch enqueued so far that it has
 * not joined yet (needed only with PS_OPT_OVERLAP; otherwise a no-op). */
int ps_join(ps_service* svc, void* stream);

/* Launches whatever PS_OPT_BATCH is holding back, without making any stream
 * wait (ps_join does both).  A caller that stops issuing rounds calls one of
 * the two; until then held-back rounds have not started. */
int ps_flush(ps_service* svc);

/* One round of the service in ONE call — what an Aggregator does when the last
 * worker's gradients of some tensors have arrived (paper Figure 1 and Section 2.1:
 * tensors become ready one layer after another during the backward pass, so a
 * round is often a few small tensors and its cost is the cost of the calls):
 * the n_push pushes of ps_push_batch, then ps_aggregate(ready, n_ready, stream),
 * then, if params_dev_ptrs_out is not NULL, the n_ready parameter pointers of
 * ps_pull_batch (in the order of `ready`).  All-or-nothing: when the aggregate is
 * rejected the pushes of this call are taken back.
 * flags: PS_ROUND_INPUTS_COMPLETE — every gradient buffer pushed for the listed
 * tasks is already complete in memory when the call is made (it arrived over the
 * network or a peer link and the host was told; nothing still enqueued on
 * `stream` writes it).  With PS_OPT_OVERLAP the launch then does not wait for
 * `stream` at all, and a round costs the host one kernel launch.  Without the
 * flag the launch is ordered after the work enqueued on `stream`, as for
 * ps_aggregate.
 * Errors: those of ps_push_batch and ps_aggregate; BAD_ARG for unknown flags. */
#define PS_ROUND_INPUTS_COMPLETE 1u
int ps_round(ps_service* svc, int n_push, const int* jobs, const int* blocks, const int* workers,
             const void* const* grad_dev_ptrs, const ps_task* ready, int n_ready, unsigned int flags,
             void* stream, const float** params_dev_ptrs_out);

/* Pull (paper Section 4): *params_dev_ptr_out receives a device pointer to the
 * block's nelem fp32 parameters.  Borrowed; stable until the block is migrated
 * or the service destroyed; contents are defined once the last ps_aggregate /
 * ps_migrate_block enqueued for the block has completed on its stream. */
int ps_pull(ps_service* svc, int job, int block, const float** params_dev_ptr_out);

/* Pull for n tasks in one call: out[i] receives the parameter pointer of
 * tasks[i] (host arrays).  All-or-nothing. */
int ps_pull_batch(ps_service* svc, const ps_task* tasks, int n, const float** params_dev_ptrs_out);

/* Pull into host memory: enqueues a device-to-host copy of the parameters on
 * `stream` (ordered after the block's last aggregate/migration). */
int ps_pull_host(ps_service* svc, int job, int block, float* params_host_dst, void* stream);

/* Moves the block's master copy — parameters, optimizer state and step
 * counter — to context `dst_ctx` (paper Section 3.2 and Appendix B: the old
 * Aggregator copies the tensor's contents to the new one, which must not
 * update it before the copy has landed).  The copy is enqueued on `stream`
 * after the block's last aggregate; later aggregates of the block wait for it;
 * the source memory is released when the copy has completed.  Pending pushes
 * stay with the block.  dst_ctx equal to the current context is a no-op.
 * Errors: BAD_ARG, NOMEM (block stays where it was), NO_DEVICE, CUDA. */
int ps_migrate_block(ps_service* svc, int job, int block, int dst_ctx, void* stream);

/* The same for n blocks at once (host array of tasks, no block listed twice), as
 * ONE batch: every destination range is reserved first (PS_ERR_NOMEM leaves all
 * blocks where they were), one gather-copy kernel moves up to 1024 blocks (96
 * where the driver refuses a parameter block above 4 KB) and one event marks
 * the batch — moving all tensors of a model costs one launch instead of one copy
 * call per tensor (the paper's Appendix B measures
 * exactly that case: the overhead of migrating all tensors of a model).
 * Errors: BAD_ARG, DUPLICATE, NOMEM, NO_DEVICE, CUDA. */
int ps_migrate_blocks(ps_service* svc, const ps_task* tasks, int n, int dst_ctx, void* stream);

/* A round that recurs.  Training is iterative (paper Section 2.2, "Iterative
 * Training"; Section 3.3.1 builds cyclic execution on it): iteration after
 * iteration the same tensors become ready in the same groups, pushed from the
 * same buffers.  ps_round_prepare records one such round — the arguments of
 * ps_round, copied — and returns a small integer; ps_round_run(round) then does
 * exactly what ps_round would do with those arguments, but the lists are already
 * resolved and, when the round's pushes are precisely the W shards of each of
 * its ready blocks, the packed task table of the previous run is reused with
 * only the step-dependent fields refreshed.  A run therefore costs the host
 * little more than the kernel launch.  Anything that could change the table
 * (a migration, ps_unregister_block, an option) makes the next run resolve and
 * build again by itself; a round whose block has been unregistered fails with
 * BAD_ARG.  params_dev_ptrs_out (may be NULL) receives the n_ready parameter
 * pointers.  ps_round_release forgets a round (its number may be handed out
 * again).  Errors of ps_round_prepare: BAD_ARG, ALIGN, DUPLICATE (task listed
 * twice).  Errors of ps_round_run: those of ps_round; all-or-nothing alike. */
int ps_round_prepare(ps_service* svc, int n_push, const int* jobs, const int* blocks, const int* workers,
                     const void* const* grad_dev_ptrs, const ps_task* ready, int n_ready, unsigned int flags,
                     int* round_out);
int ps_round_run(ps_service* svc, int round, void* stream, const float** params_dev_ptrs_out);
int ps_round_release(ps_service* svc, int round);

/* Per-block statistics of the last aggregate (paper Section 3.1: profilers feed
 * the manager): squared norm of the aggregated gradient and the step counter.
 * Waits for the block's last aggregate to finish.  Either out pointer may be
 * NULL.  Before the first aggregate the norm is 0 and the step 0. */
int ps_block_stats(ps_service* svc, int job, int block, double* grad_sqnorm_out,
                   unsigned long long* step_out);

/* Device time of the block's last aggregate, recorded when PS_OPT_PROFILE was on
 * for that launch (zeros otherwise) — the counterpart of the per-task execution
 * time e_t that the paper's profilers collect for the assignment scheme
 * (Section 3.1; Pseudocode 1 takes e_t as input).  busy = sum over the task's
 * chunks of the time a CTA spent on the chunk (CTA-microseconds; chunks of one
 * task run concurrently on many CTAs); span = last chunk end - first chunk
 * start.  Timer: the GPU's %globaltimer (resolution is device dependent, up to
 * about 1 us).  Waits for the block's last aggregate.  Out pointers may be NULL. */
int ps_block_profile(ps_service* svc, int job, int block, double* busy_us_out, double* span_us_out);

/* The same over all blocks of a job (each block's last aggregate): summed busy
 * time, span from the earliest chunk start to the latest chunk end, and the
 * number of blocks that carried a profile. */
int ps_job_profile(ps_service* svc, int job, double* busy_us_out, double* span_us_out, int* blocks_out);

/* Device pointers to the block's optimizer state (momentum | Adam m, and
 * Adam v or NULL) and its current context; for tests and checkpoints. */
int ps_block_state(ps_service* svc, int job, int block, const float** state0_dev_ptr_out,
                   const float** state1_dev_ptr_out, int* ctx_out);

/* One (job, block, chunk) descriptor as the kernel will see it. */
typedef struct {
  int job, block;
  unsigned long long elem_begin, elem_count;
  int num_workers;
  int vector_path; /* 1 if every pointer of the task allows 128-bit accesses */
} ps_chunk_info;

/* Builds the packed task table for `ready` exactly as ps_aggregate would,
 * without launching or consuming anything, and writes up to `cap` chunk
 * descriptors (in the order CTAs will claim them) to `out` (host, may be NULL);
 * *n_chunks_out receives the total.  Works on planning-only services.
 * Errors as ps_aggregate's validation. */
int ps_plan(ps_service* svc, const ps_task* ready, int n_ready, ps_chunk_info* out, size_t cap,
            size_t* n_chunks_out);

int ps_set_option(ps_service* svc, int option, long long value);
int ps_get_option(ps_service* svc, int option, long long* value_out);

/* Bytes in use / largest free range of a context's arena. */
int ps_arena_info(ps_service* svc, int ctx, size_t* used_out, size_t* largest_free_out);

/* Size of the registry: registered jobs, registered blocks, and entries of the
 * block table (registered blocks plus entries that ps_unregister_block released
 * and a later ps_register_block will use again — the table does not grow while
 * blocks come and go). */
int ps_registry_info(ps_service* svc, size_t* jobs_out, size_t* blocks_out, size_t* block_entries_out);

/* Number of aggregation kernels launched so far and the grid/block size and
 * variant name of the last one (for launch accounting in benchmarks). */
int ps_launch_info(ps_service* svc, unsigned long long* launches_out, int* grid_out, int* block_out,
                   const char** kernel_name_out);

/* Launch accounting per kernel variant (0 = persistent direct-load kernel,
 * 1 = small-launch kernel with the table in its parameters, 2 = bulk-copy ring):
 * launches so far, the algorithmic bytes they covered (W shards read, parameters
 * and state read and written, dense semantics) and the kernel's name.
 * Errors: BAD_ARG (variant out of range). */
int ps_launch_stats(ps_service* svc, int variant, unsigned long long* launches_out,
                    unsigned long long* algorithmic_bytes_out, const char** kernel_name_out);

/* Waits for the device and reports the kernels' status word: 0 = no fault;
 * non-zero = a bounded wait inside a kernel expired (the launch returned early
 * and its results are undefined). */
int ps_device_status(ps_service* svc, int* status_out);

/* Largest block ps_aggregate_block_noalloc accepts (2^24 elements). */
#define PS_NOALLOC_MAX_ELEMS ((size_t)1 << 24)

/* Aggregates ONE block without allocating anything, for callers that must not
 * touch the allocator.  (The paper has no counterpart: this is a convenience of
 * this library.)  Typical callers: a process whose framework has already
 * reserved all device memory for its own pool, so a cudaMalloc here could fail
 * or fragment it; a latency-critical loop that cannot take the implicit
 * device-wide synchronisation an allocation may cause; code that runs where the
 * memory budget is fixed at start-up.  No ps_service is involved: the caller
 * owns and passes everything —
 *   job                hyper-parameters (host pointer; W = job->num_workers)
 *   step               t >= 1, the number of this aggregate for the block
 *   nelem              1 .. PS_NOALLOC_MAX_ELEMS, else PS_ERR_TOO_LARGE
 *   params/state0/state1   device pointers to nelem floats, updated in place
 *                      (state1 = Adam's second moment, NULL for SGD)
 *   shard_dev_ptrs     host array of W device pointers to the gradient shards
 *   sqnorm_dev_out     device pointer that receives sum G*G, or NULL
 * and gets the same arithmetic as ps_aggregate (same kernel).  The work is
 * enqueued on `stream` of the CURRENT device; nothing is waited for.
 *
 * The kernel's scratch (task table, work counter, per-chunk partial sums: 20 KB)
 * lives in a fixed array inside the library's device image, so every GPU that
 * loads the library holds those 20 KB until the process exits.  The first call
 * on a device looks the array's address up and caches it; make that first call
 * outside any stream capture.  All calls on a device share the array and each
 * call re-initialises the parts that must start at zero, so calls must not
 * overlap on the GPU: issue them on one stream, or order the streams yourself.
 * Calls cudaMalloc/cudaFree never.  Errors: BAD_ARG, ALIGN (a pointer not
 * 4-byte / element aligned), TOO_LARGE, CUDA. */
int ps_aggregate_block_noalloc(const ps_job_desc* job, unsigned long long step, size_t nelem,
                               float* params_dev, float* state0_dev, float* state1_dev_or_null,
                               const void* const* shard_dev_ptrs, double* sqnorm_dev_out_or_null,
                               void* stream);

/* Migration between two services (the paper's migration between Aggregator
 * machines, Section 3.2 and Appendix B: the old Aggregator copies the tensor's
 * contents and metadata to the new one, which must not update the tensor before
 * the copy has landed).  ps_migrate_block moves a block between contexts of ONE
 * service; these three calls move it between services, e.g. between the GPUs of
 * a block-sharded deployment, through any device memory both can address (a
 * peer buffer):
 *
 *   ps_block_export  enqueues on `stream`, after the block's last aggregate, a
 *       copy of its packed state into dst_dev: parameters | state0 | (state1),
 *       each section round_up(4*nelem, 256) bytes — *bytes_out in total — and
 *       reports the block's step counter.  dst_dev == NULL only reports the two
 *       numbers.  The service is unchanged; pending pushes are not exported.
 *   ps_block_import  for a block registered here (same nelem, same optimizer):
 *       enqueues on `stream` the copy of such a packed state into the block's
 *       range and sets its step counter.  Later aggregates of the block wait for
 *       the copy (they are ordered after it whatever their stream); pushes may
 *       arrive meanwhile.  src_bytes must equal the block's packed size.
 *   ps_unregister_block  waits (host) for the work this service enqueued for
 *       the block, releases its arena range and staging buffer and forgets the
 *       id, which may be registered again.  Pending pushes are dropped.
 * The caller orders the two sides: the export's stream has reached the copy's
 * end before the importer's copy starts (same process: an event; two
 * processes: synchronize, then a host barrier).
 * Errors: BAD_ARG (unknown block, dst too small, size mismatch), NO_DEVICE, CUDA. */
int ps_block_export(ps_service* svc, int job, int block, void* dst_dev, size_t dst_cap, size_t* bytes_out,
                    unsigned long long* step_out, void* stream);
int ps_block_import(ps_service* svc, int job, int block, const void* src_dev, size_t src_bytes,
                    unsigned long long step, void* stream);
int ps_unregister_block(ps_service* svc, int job, int block);

/* ---------------------------------------------------------------------------
 * Peer buffers: several Aggregators on the GPUs of one node.
 *
 * The paper spreads the tensors of a job over several Aggregator machines that
 * exchange nothing but migrated tensors (Section 3.2).  On one node the
 * counterpart is one service per GPU, one process each, every block owned by
 * one of them; there is no collective in the aggregation path.  A worker's
 * gradient shards then sit in another process's (often another GPU's) memory:
 * the worker's process allocates them with ps_peer_alloc and passes the 64-byte
 * handle to the owners by any host channel, an owner maps the buffer with
 * ps_peer_open and gives the mapped address (plus the shard's offset) to
 * ps_push.  The aggregation kernel reads it in place with ordinary loads: over
 * NVLink when the GPUs differ, with no staging copy.
 *
 *   ps_peer_alloc  allocates `bytes` of device memory on `device` (its own
 *                  allocation, 256-byte aligned) and writes its handle.
 *                  Owner: the caller, until ps_peer_free.
 *   ps_peer_open   maps a buffer exported by ANOTHER process into this one for
 *                  use on `device` (peer access is enabled as needed); the
 *                  mapping is read/write and stays valid until ps_peer_close or
 *                  until the exporter frees the buffer, whichever comes first —
 *                  the exporter must outlive every use.  Opening a handle in
 *                  the process that exported it is an error (use the pointer).
 * Errors: BAD_ARG, NOMEM, CUDA (text: ps_peer_last_error, per host thread).
 * Ordering between the processes (the worker has finished writing a shard
 * before the owner's launch reads it; the owner's launch has completed before
 * the worker overwrites it) is the callers' business: a host barrier after a
 * stream synchronize on each side is enough.
 * ------------------------------------------------------------------------- */
#define PS_PEER_HANDLE_BYTES 64
int ps_peer_alloc(int device, size_t bytes, void** dev_ptr_out, unsigned char* handle_out);
int ps_peer_free(int device, void* dev_ptr);
int ps_peer_open(int device, const unsigned char* handle, void** dev_ptr_out);
int ps_peer_close(int device, void* dev_ptr);
const char* ps_peer_last_error(void);

/* Ordering between processes WITHOUT a host wait: interprocess events.  One
 * process creates an event and passes its 64-byte handle on; the others open
 * it.  ps_peer_event_record(event, stream) marks a point of the recorder's
 * stream; ps_peer_event_wait(event, stream) makes a stream of any process wait
 * for the most recent record — which must already have been ISSUED when the
 * wait is enqueued (a wait on an event that nobody has recorded yet passes at
 * once), so the waiter learns over a host channel that the record call has been
 * made; it does not have to learn that the device has reached it.  Used for
 * migration between services (the new owner's copy waits for the old owner's;
 * paper Appendix B, "Data Consistency") and for staged pushes (the owner's
 * aggregate waits for the workers' copies into its memory).  Events are
 * destroyed by every process that holds them.
 * ps_peer_copy_many enqueues n plain copies (copy engines) on `stream`;
 * either side of each may be mapped peer memory.
 * Errors: BAD_ARG, CUDA (text: ps_peer_last_error). */
int ps_peer_event_create(int device, void** event_out, unsigned char* handle_out);
int ps_peer_event_open(int device, const unsigned char* handle, void** event_out);
int ps_peer_event_record(void* event, void* stream);
int ps_peer_event_wait(void* event, void* stream);
int ps_peer_event_destroy(void* event);
int ps_peer_copy_many(int n, void* const* dsts, const void* const* srcs, const size_t* bytes, void* stream);

/* Pull from another process (paper Section 4: Pull returns the current
 * parameters of (job, tensor)).  ps_arena_export writes the handle of a
 * context's arena, which a worker process maps with ps_peer_open;
 * ps_block_location says where in that arena a block lives: its parameters are
 * the nelem floats at `offset`, its optimizer state follows in sections of
 * `section` bytes.  The location changes when the block migrates; the contents
 * are defined once the owner's last aggregate of the block has completed (the
 * processes order that between themselves, as for peer buffers).  The mapping
 * is for reading: a writer other than the owner's kernels breaks the service.
 * Errors: BAD_ARG, NO_DEVICE, CUDA. */
int ps_arena_export(ps_service* svc, int ctx, unsigned char* handle_out, size_t* bytes_out);
int ps_block_location(ps_service* svc, int job, int block, int* ctx_out, size_t* offset_out,
                      size_t* section_bytes_out);

/* ---------------------------------------------------------------------------
 * Planner: which Aggregator (context) runs which aggregation task.  Host only.
 *
 * The paper's assignment heuristic — Section 3.3.1, Pseudocode 1 "Model
 * Aggregation Assignment Scheme" — with cyclic execution: an Aggregator's cycle
 * C_n is the largest iteration duration D_j among its jobs; job j gets a slot
 * every d_j = max(D_j, C_n / floor(C_n / D_j)); a destination is dropped when a
 * job on it (or the new task's job) would lose (d_j - D_j)/d_j >= loss_limit;
 * among the rest the task goes to the best fit, i.e. the Aggregator with the
 * fewest free slots F_n = C_n - sum_j floor(C_n/d_j) * sum_{t of j on n} e_t that
 * still hold the task's floor(C_n/d_k) * e_t; if none, a new Aggregator is
 * allocated.  Times are in any one unit (e.g. microseconds from
 * ps_block_profile for e_t, the job's measured iteration period for D_j).
 * Aggregator indices count from 0 and are meant to be used as `ctx` in
 * ps_register_block / ps_migrate_block.
 * ------------------------------------------------------------------------- */
typedef struct ps_planner ps_planner; /* opaque */

/* loss_limit: the paper's LossLimit (default 0.1), in (0, 1]. */
int ps_planner_create(ps_planner** out, double loss_limit);
int ps_planner_destroy(ps_planner* pl);
/* Registers a job with profiled iteration duration D_j > 0. */
int ps_planner_add_job(ps_planner* pl, double iter_duration, int* job_out);
/* Pseudocode 1 for one new task of `job` with execution time e_t > 0: chooses
 * (or allocates) an Aggregator and records the assignment. */
int ps_planner_assign(ps_planner* pl, int job, double exec_time, int* task_out, int* aggregator_out);
/* Job exit (Section 3.3.2): drops the job's tasks, releases Aggregators left
 * empty, then repeatedly tries to empty the least-loaded Aggregator by
 * re-assigning its tasks to the others without new allocations; stops at the
 * first one that cannot be emptied (its tasks stay).  Released Aggregators keep
 * their index and are never reused.  Tasks that moved report their new
 * Aggregator through ps_planner_task_info (the caller migrates the blocks). */
int ps_planner_remove_job(ps_planner* pl, int job, int* released_out);
int ps_planner_task_info(ps_planner* pl, int task, int* job_out, int* aggregator_out, double* exec_time_out);
/* Cyclic execution (Section 3.3.1): how many times the task runs in one cycle of
 * its Aggregator, floor(C_n / d_j), and the period d_j of its slots there. */
int ps_planner_task_runs(ps_planner* pl, int task, int* runs_per_cycle_out, double* slot_period_out);
/* cycle = C_n; load = W_n = sum_j floor(C_n/d_j) * sum e_t (Appendix C). */
int ps_planner_aggregator_info(ps_planner* pl, int aggregator, int* alive_out, double* cycle_out,
                               double* load_out, int* num_tasks_out);
/* D_j, the current d_j (largest over the Aggregators that hold its tasks) and
 * the loss (d_j - D_j)/d_j. */
int ps_planner_job_info(ps_planner* pl, int job, double* profiled_out, double* current_out, double* loss_out);
int ps_planner_num_aggregators(ps_planner* pl, int* allocated_out, int* alive_out);
/* Late request ("Handling Outliers in Cyclic Execution"): returns 1 if a request
 * of `exec_time` that missed its slot still fits the current cycle after the
 * `remaining_scheduled` time of the requests still due in it is reserved, 0 if
 * it has to wait for the next cycle. */
int ps_planner_outlier_fits(double cycle, double now_in_cycle, double remaining_scheduled, double exec_time);

const char* ps_strerror(int status);
/* Text of the last CUDA error seen by this service ("" if none). */
const char* ps_last_cuda_error(ps_service* svc);
const char* ps_version(void);

#ifdef __cplusplus
}
#endif
#endif /* PS_B200_H */
