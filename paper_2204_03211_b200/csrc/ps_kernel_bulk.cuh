// Aggregation kernel, bulk-copy variant for sm_100a: one persistent CTA per SM,
// warp-specialised.  A producer warp claims (job, block, chunk) work items from
// the table's atomic counter, cuts each chunk into tiles of 4096 elements and
// streams every tile into a shared-memory ring with 1-D bulk asynchronous
// copies (TMA unit, completion counted on an mbarrier; every CTA fetches its own
// tiles, no multicast).  A tile is cut ALONG THE WORKERS: one ring stage holds
// the tile's rows of a few consecutive workers (three fp32 or six bf16 shards,
// 16 KB or 8 KB per row: issuing a copy costs the producer about a hundred
// cycles whatever its size, so copies are made large), the next stage the next
// workers, and the parameters and optimizer state ride in the tile's last
// stage.  Eight consumer warps keep the running sums of a tile in registers
// across its stages — worker order 0..W-1, binary32, so the bits are those of
// the direct-load kernel — and on the last stage apply the optimizer and store
// parameters and state with 128-bit stores.  The ring keeps 192 KB per SM in
// flight whatever W is.  A tenth warp collects each finished chunk's partial
// sums of squares and draws the tickets that count a task's chunks once per
// eight chunks: done by the producer, per chunk, those round trips to memory
// and their fences were the kernel's bottleneck — the producer has about a
// thousand cycles per stage to keep the ring full.
//
// Chunks that cannot use bulk copies (a shard pointer that is not 16-byte
// aligned, fewer elements than one vector) are handed to the consumers as
// "direct" work and read with ordinary loads.  Warps synchronise through
// mbarriers only (never a CTA-wide barrier between set-up and exit), and every
// mbarrier wait is bounded by the table's limit: on expiry the warp records an
// error code in the device status word and stops; before the CTA leaves, the
// producer waits (with a generous limit of its own) for its copies in flight.
#pragma once

#include "ps_math.cuh"

namespace psb {

constexpr int kBulkConsumerWarps = 8;
constexpr int kBulkConsumers = kBulkConsumerWarps * 32;     // 256 consumer threads
constexpr int kBulkThreads = kBulkConsumers + 64;           // + one producer warp + one publisher warp
constexpr int kPubSlots = 8;                                // finished chunks waiting for the publisher
constexpr unsigned int kPubEnd = 0xffffffffu;               // in place of a task: no more chunks from this CTA
constexpr int kPubRuns = 8;                                 // chunks a CTA collects before it draws their tasks' tickets
constexpr int kStageBytes = 49152;
constexpr int kStages = 4;
constexpr int kBulkSmemBytes = kStages * kStageBytes + 1024;
constexpr unsigned int kRingTile = 4096;                    // elements per tile: 16 per consumer thread
static_assert(3u * kRingTile * 4u <= (unsigned int)kStageBytes, "a stage holds p and two state rows of a tile");
constexpr long long kDrainCycles = 4000000000ll;            // limit of the producer's own wait for its copies (about 2 s)
constexpr unsigned int kWaitUnit = 1024;                    // the table gives its wait limit in units of this many cycles

enum : unsigned int { kTileFirst = 1u, kTileLast = 2u, kTileDirect = 4u, kTileEnd = 8u, kChunkEnd = 16u };

// What the consumers need to know about one ring stage; written by the producer
// before it arms the stage's barrier.
struct StageMeta {
  float* p;
  float* s0;
  float* s1;
  unsigned long long e0;               // first element of the tile inside its block
  unsigned int task, chunk;
  unsigned int cnt;                    // elements of the tile (a multiple of the vector width)
  unsigned int nrows;                  // shard rows in this stage
  unsigned int state_off;              // byte offset of the p row (kTileLast), rows of kRingTile floats follow
  unsigned int flags;
  unsigned int pub_slot;               // kChunkEnd: where the chunk's partial sums go
  int W, kind;                         // kind = (optimizer << 1) | gradient type
  Hp h;
};

// ---- PTX wrappers ----------------------------------------------------------

__device__ __forceinline__ unsigned int smem_u32(const void* p) {
  return static_cast<unsigned int>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(unsigned long long* bar, unsigned int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned long long* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(unsigned long long* bar, unsigned int bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned long long* bar, unsigned int parity) {
  unsigned int ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_test_wait(unsigned long long* bar, unsigned int parity) {
  unsigned int ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false if the limit (in cycles) expired or another warp aborted.
// try_wait may itself suspend the thread for a while (a hardware time-out that is not ours
// to set), so limits below about a millisecond are kept with the non-blocking test instead.
__device__ __forceinline__ bool mbar_wait(unsigned long long* bar, unsigned int parity, volatile int* abort_flag,
                                          long long limit) {
  const bool quick = limit < (1ll << 20);
  if (quick ? mbar_test_wait(bar, parity) : mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  unsigned int spins = 0;
  while (!(quick ? mbar_test_wait(bar, parity) : mbar_try_wait(bar, parity))) {
    if (quick || (++spins & 15u) == 0) {
      if (*abort_flag) return false;
      if (clock64() - t0 > limit) return false;
    }
  }
  return true;
}
// 1-D bulk copy global -> this CTA's shared memory, completion on `bar`.
// Both addresses 16-byte aligned, size a multiple of 16 bytes.
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, unsigned int bytes, unsigned long long* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

// ---- consumer bodies ------------------------------------------------------------

// Adds the stage's shard rows to the thread's running sums.  A thread owns the
// 16-byte groups c, c + 256, ... of every row: four groups of four fp32 elements,
// or two groups of eight bf16 elements — 16 elements of the tile either way.
template <bool BF16>
__device__ __forceinline__ void ring_accumulate(unsigned int c, const unsigned char* __restrict__ st, unsigned int nrows,
                                                unsigned int cnt, bool first, float (&acc)[16]) {
  constexpr int G = BF16 ? 2 : 4;
  constexpr unsigned int kRow = kRingTile * (BF16 ? 2u : 4u);
  const unsigned int ng = cnt >> (BF16 ? 3 : 2);
  bool act[G];
#pragma unroll
  for (int j = 0; j < G; ++j) act[j] = c + (unsigned int)j * kBulkConsumers < ng;
#pragma unroll 2
  for (unsigned int r = 0; r < nrows; ++r) {
    const uint4* row = reinterpret_cast<const uint4*>(st + (size_t)r * kRow);
    uint4 x[G];
#pragma unroll
    for (int j = 0; j < G; ++j) x[j] = act[j] ? row[c + (unsigned int)j * kBulkConsumers] : make_uint4(0, 0, 0, 0);
    if (first && r == 0) {
#pragma unroll
      for (int j = 0; j < G; ++j) {
        if (BF16) {
          acc[8 * j + 0] = bf16_lo(x[j].x); acc[8 * j + 1] = bf16_hi(x[j].x);
          acc[8 * j + 2] = bf16_lo(x[j].y); acc[8 * j + 3] = bf16_hi(x[j].y);
          acc[8 * j + 4] = bf16_lo(x[j].z); acc[8 * j + 5] = bf16_hi(x[j].z);
          acc[8 * j + 6] = bf16_lo(x[j].w); acc[8 * j + 7] = bf16_hi(x[j].w);
        } else {
          acc[4 * j + 0] = __uint_as_float(x[j].x); acc[4 * j + 1] = __uint_as_float(x[j].y);
          acc[4 * j + 2] = __uint_as_float(x[j].z); acc[4 * j + 3] = __uint_as_float(x[j].w);
        }
      }
    } else {
#pragma unroll
      for (int j = 0; j < G; ++j) {
        if (BF16) {
          add_bf16x2(acc[8 * j + 0], acc[8 * j + 1], x[j].x);
          add_bf16x2(acc[8 * j + 2], acc[8 * j + 3], x[j].y);
          add_bf16x2(acc[8 * j + 4], acc[8 * j + 5], x[j].z);
          add_bf16x2(acc[8 * j + 6], acc[8 * j + 7], x[j].w);
        } else {
          acc[4 * j + 0] = __fadd_rn(acc[4 * j + 0], __uint_as_float(x[j].x));
          acc[4 * j + 1] = __fadd_rn(acc[4 * j + 1], __uint_as_float(x[j].y));
          acc[4 * j + 2] = __fadd_rn(acc[4 * j + 2], __uint_as_float(x[j].z));
          acc[4 * j + 3] = __fadd_rn(acc[4 * j + 3], __uint_as_float(x[j].w));
        }
      }
    }
  }
}

// The tile's last stage: parameters and state come out of the ring, the update goes to global memory.
template <int OPT, bool BF16>
__device__ __forceinline__ void ring_update(unsigned int c, const StageMeta& m, const unsigned char* __restrict__ st,
                                            const float (&acc)[16], double& sq) {
  const float4* rp = reinterpret_cast<const float4*>(st + m.state_off);
  const float4* ra = rp + kRingTile / 4;
  const float4* rb = ra + kRingTile / 4;
  const unsigned int ng4 = m.cnt >> 2;
  const float4 z = make_float4(0, 0, 0, 0);
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    // fp32: float4 group c + 256 q.  bf16: the thread's 16-byte group c + 256 (q / 2) holds the
    // float4 groups 2 (c + 256 (q / 2)) and the next one.
    const unsigned int g = BF16 ? 2u * (c + (unsigned int)(q >> 1) * kBulkConsumers) + (unsigned int)(q & 1)
                                : c + (unsigned int)q * kBulkConsumers;
    if (g < ng4)
      update4<OPT>(m.h, make_float4(acc[4 * q], acc[4 * q + 1], acc[4 * q + 2], acc[4 * q + 3]), m.p, m.s0, m.s1,
                   (size_t)m.e0 + 4 * (size_t)g, rp[g], ra[g], OPT == 1 ? rb[g] : z, sq);
  }
}

// ---- the kernel ----------------------------------------------------------------

__global__ void __launch_bounds__(kBulkThreads, 1)
ps_aggregate_bulk_kernel(unsigned char* __restrict__ table, const PsJobDev* __restrict__ jobs,
                         PsStat* __restrict__ stats, double* __restrict__ partials, int* __restrict__ status,
                         unsigned long long* done_word, unsigned long long seq) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* ring = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127);
  __shared__ __align__(8) unsigned long long full_bar[kStages];
  __shared__ __align__(8) unsigned long long empty_bar[kStages];
  __shared__ __align__(16) StageMeta meta[kStages];
  __shared__ __align__(8) unsigned long long pub_bar[kPubSlots];
  __shared__ double s_part[kPubSlots][kBulkConsumerWarps];   // a chunk's sums of squares, one per consumer warp
  __shared__ unsigned int s_pub_task[kPubSlots], s_pub_chunk[kPubSlots];
  __shared__ unsigned int s_pub_done;      // chunks published so far (written by the publisher)
  __shared__ unsigned int s_run_task[kPubRuns], s_run_chunks[kPubRuns];
  __shared__ int s_abort;

  PsTableHdr* hdr = reinterpret_cast<PsTableHdr*>(table);
  PsTaskDev* tasks = reinterpret_cast<PsTaskDev*>(table + hdr->tasks_off);
  const unsigned int* starts = reinterpret_cast<const unsigned int*>(table + hdr->starts_off);
  const void* const* ptrs = reinterpret_cast<const void* const*>(table + hdr->ptrs_off);
  const unsigned int n_tasks = hdr->n_tasks, total = hdr->total_chunks;
  const long long wait_limit = (long long)hdr->wait_units * kWaitUnit;

  const unsigned int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&full_bar[s], 1);                       // the producer's arrive (+ transaction bytes)
      mbar_init(&empty_bar[s], kBulkConsumerWarps);     // one arrive per consumer warp
    }
    for (int s = 0; s < kPubSlots; ++s) mbar_init(&pub_bar[s], kBulkConsumerWarps);
    s_pub_done = 0;
    s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();

  if (warp == kBulkConsumerWarps) {
    // ------------------------------------------------------------ producer warp
    unsigned int cursor = 0, stage = 0, fills = 0;   // fills: stages posted so far
    unsigned int pend_mask = 0, pend_par = 0;        // stages whose last fill carried copies, and its parity
    unsigned int closed = 0;                         // chunks this CTA has closed (their last stage posted)
    bool ok = true;
    unsigned int idx = 0, next = 0;
    if (lane == 0) idx = atomicAdd(&hdr->counter, 1u);
    idx = __shfl_sync(0xffffffffu, idx, 0);

    // what every stage of a chunk repeats, read from the table once per chunk
    struct ChunkCtx {
      Hp h;
      float *p, *s0, *s1;
      const void* const* shards;
      int W, kind;
      unsigned int ges, nstate_rows;
    } cc = {};

    // A finished chunk's partial sums go to slot closed % kPubSlots: free once the publisher is
    // fewer than kPubSlots chunks behind (it normally is: a publish costs a few microseconds,
    // a chunk several).
    auto slot_free = [&]() {
      const volatile unsigned int* pd = &s_pub_done;
      if (closed - *pd >= (unsigned int)kPubSlots) {
        const long long t0 = clock64();
        while (closed - *pd >= (unsigned int)kPubSlots) {
          if (*const_cast<volatile int*>(&s_abort) || clock64() - t0 > wait_limit) { ok = false; break; }
        }
      }
      ok = __all_sync(0xffffffffu, ok);
      return ok;
    };

    // Posts one stage: waits for the slot, writes its description, arms the barrier and
    // issues the copies (lane l fetches row l of the stage): nsh shard rows from worker
    // `first_w`, then the state rows if this is the tile's last stage.
    auto post = [&](unsigned int task, unsigned int chunk, size_t e0,
                    unsigned int cnt, unsigned int first_w, unsigned int nsh, bool with_state, unsigned int flags) {
      const unsigned int use = fills / kStages;
      if (use > 0) ok = mbar_wait(&empty_bar[stage], (use - 1) & 1u, &s_abort, wait_limit);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) return;
      if ((flags & kChunkEnd) && !slot_free()) return;
      const unsigned int ges = cc.ges;
      const unsigned int nst = with_state ? cc.nstate_rows : 0u;
      const unsigned int row_slot = kRingTile * ges;
      unsigned char* dst = ring + (size_t)stage * kStageBytes;
      const unsigned int bytes = cnt * (nsh * ges + nst * 4u);
      if (lane == 0) {
        StageMeta& m = meta[stage];
        m.p = cc.p; m.s0 = cc.s0; m.s1 = cc.s1;
        m.e0 = e0;
        m.task = task; m.chunk = chunk; m.cnt = cnt; m.nrows = nsh;
        m.state_off = nsh * row_slot;
        m.flags = flags;
        m.pub_slot = closed % (unsigned int)kPubSlots;
        m.W = cc.W;
        m.kind = cc.kind;
        m.h = cc.h;
        if (flags & kChunkEnd) {
          s_pub_task[m.pub_slot] = task;
          s_pub_chunk[m.pub_slot] = chunk;
        }
        if (bytes) mbar_arrive_expect_tx(&full_bar[stage], bytes);
        else mbar_arrive(&full_bar[stage]);
      }
      if (flags & kChunkEnd) ++closed;
      __syncwarp();
      if (bytes) {
        if (lane < nsh) {
          const unsigned char* src = static_cast<const unsigned char*>(ld_ptr(cc.shards, (int)(first_w + lane))) + e0 * ges;
          bulk_g2s(dst + (size_t)lane * row_slot, src, cnt * ges, &full_bar[stage]);
        } else if (lane < nsh + nst) {
          const unsigned int q = lane - nsh;
          const float* src = (q == 0 ? cc.p : (q == 1 ? cc.s0 : cc.s1)) + e0;
          bulk_g2s(dst + (size_t)nsh * row_slot + (size_t)q * kRingTile * 4, src, cnt * 4, &full_bar[stage]);
        }
        pend_mask |= 1u << stage;
        pend_par = (pend_par & ~(1u << stage)) | ((use & 1u) << stage);
      } else {
        pend_mask &= ~(1u << stage);
      }
      ++fills;
      stage = (stage + 1 == kStages) ? 0 : stage + 1;
    };

    // What the producer reads from a task's record.  The record of the NEXT chunk's task is
    // requested while the current chunk streams (its claim is issued at the top of the chunk):
    // found and read only when the chunk starts, the table look-ups — a chain of three or four
    // dependent trips to L2 — kept the producer busy for a third of a W = 4 chunk.
    struct TaskRegs {
      float *p, *s0, *s1;
      unsigned long long nelem;
      unsigned int shard_row, first_chunk, vec_ok, tile_elems, chunk_elems;
      int job;
      float ss_t, sbc2_t;
    };
    auto load_task = [&](unsigned int t) {
      const PsTaskDev* T = tasks + t;
      TaskRegs r;
      r.p = T->p; r.s0 = T->s0; r.s1 = T->s1;
      r.nelem = T->nelem;
      r.shard_row = T->shard_row; r.first_chunk = T->first_chunk;
      r.vec_ok = T->vec_ok; r.tile_elems = T->tile_elems; r.chunk_elems = T->chunk_elems;
      r.job = T->job;
      r.ss_t = T->ss_t; r.sbc2_t = T->sbc2_t;
      return r;
    };
    TaskRegs tr = {}, ntr = {};
    unsigned int ncursor = 0;
    bool looked = true;
    auto look_ahead = [&]() {            // once per chunk, after its first stages are on their way
      if (looked) return;
      looked = true;
      next = __shfl_sync(0xffffffffu, next, 0);
      ncursor = cursor;
      ntr = tr;
      if (next < total) {
        ncursor = find_task(starts, n_tasks, cursor, next, lane);
        if (ncursor != cursor) ntr = load_task(ncursor);
      }
    };
    if (idx < total) {
      cursor = find_task(starts, n_tasks, cursor, idx, lane);
      tr = load_task(cursor);
    }

    while (ok && idx < total) {
      if (lane == 0) next = atomicAdd(&hdr->counter, 1u);      // overlaps this chunk's copies
      looked = false;
      const PsJobDev* J = jobs + tr.job;
      const unsigned int W = (unsigned int)J->W;
      const unsigned int ges = J->grad_dtype ? 2u : 4u;
      const unsigned int vecw = J->grad_dtype ? 8u : 4u;
      const unsigned int state_bytes = (J->opt ? 3u : 2u) * kRingTile * 4u;
      const unsigned int rows_per_stage = kStageBytes / (kRingTile * ges);
      const unsigned int chunk_elems = tr.chunk_elems;
      const size_t begin = (size_t)(idx - tr.first_chunk) * chunk_elems;
      const unsigned int count = (unsigned int)min((unsigned long long)chunk_elems, tr.nelem - begin);
      const unsigned int body = count & ~(vecw - 1);
      cc.h.lr = J->lr; cc.h.mom = J->mom; cc.h.wd = J->wd; cc.h.b1 = J->b1; cc.h.b2 = J->b2;
      cc.h.omb1 = J->omb1; cc.h.omb2 = J->omb2; cc.h.eps = J->eps; cc.h.gs = J->gs;
      cc.h.ss_t = tr.ss_t; cc.h.sbc2_t = tr.sbc2_t;
      cc.p = tr.p; cc.s0 = tr.s0; cc.s1 = tr.s1;
      cc.shards = ptrs + tr.shard_row;
      cc.W = J->W;
      cc.kind = (J->opt << 1) | J->grad_dtype;
      cc.ges = ges;
      cc.nstate_rows = J->opt ? 3u : 2u;
      if (tr.tile_elems == 0 || tr.vec_ok == 0 || body == 0) {
        post(cursor, idx, begin, 0u, 0u, 0u, false, kTileDirect | kChunkEnd);
      } else {
        for (unsigned int off = 0; ok && off < body; off += kRingTile) {
          const unsigned int cnt = min(kRingTile, body - off);
          const unsigned int end_flag = (off + kRingTile >= body) ? kChunkEnd : 0u;
          for (unsigned int w = 0; ok && w < W;) {
            const unsigned int nsh = min(rows_per_stage, W - w);
            const bool last_rows = w + nsh == W;
            const bool with_state = last_rows && nsh * kRingTile * ges + state_bytes <= (unsigned int)kStageBytes;
            post(cursor, idx, begin + off, cnt, w, nsh, with_state,
                 (w == 0 ? kTileFirst : 0u) | (with_state ? (kTileLast | end_flag) : 0u));
            w += nsh;
            if (ok && last_rows && !with_state)       // the state rows get a stage of their own
              post(cursor, idx, begin + off, cnt, W, 0u, true, kTileLast | end_flag);
            look_ahead();
          }
        }
      }
      look_ahead();
      idx = next;
      cursor = ncursor;
      tr = ntr;
    }
    // end marker for the consumers; the publisher learns how many chunks to expect
    if (ok) {
      const unsigned int use = fills / kStages;
      if (use > 0) ok = mbar_wait(&empty_bar[stage], (use - 1) & 1u, &s_abort, wait_limit);
      ok = __all_sync(0xffffffffu, ok);
      if (ok && lane == 0) {
        meta[stage].flags = kTileEnd;
        mbar_arrive(&full_bar[stage]);
      }
      // and for the publisher: a slot whose task is the end mark, armed in the consumers' stead
      if (ok && slot_free()) {
        const unsigned int slot = closed % (unsigned int)kPubSlots;
        if (lane == 0) s_pub_task[slot] = kPubEnd;
        __syncwarp();
        if (lane < kBulkConsumerWarps) mbar_arrive(&pub_bar[slot]);
      }
    }
    if (!ok && lane == 0) {
      // an expired wait (here or in a consumer): flag it, then let this CTA's own copies land
      // before the CTA and its shared memory go away
      s_abort = 1;
      atomicExch(status, 1);
      for (int s = 0; s < kStages; ++s)
        if ((pend_mask >> s) & 1u) {
          const long long t0 = clock64();
          while (!mbar_try_wait(&full_bar[s], (pend_par >> s) & 1u) && clock64() - t0 < kDrainCycles) {}
        }
    }
    __syncwarp();
  } else if (warp == kBulkConsumerWarps + 1) {
    // ------------------------------------------------------------ publisher warp
    // Chunk k of this CTA leaves its eight partial sums in slot k % kPubSlots; each consumer
    // warp arrives on the slot's barrier once its share is there.  This warp copies them to
    // global memory and remembers which task they belong to.  The tickets that count a
    // task's chunks — and with them the fences — are drawn once per kPubRuns chunks (and
    // when the CTA runs out of work): a memory fence executed by ANY warp of the SM while
    // bulk copies are in flight slows the ring down (10 % of its throughput with two
    // fences per chunk, measured with the fences here, in the producer, and left out).
    // Whoever draws a task's last ticket adds its partial sums up in a fixed order; doing
    // all of that at the CTA's end instead would leave the sums of most tasks to the few
    // CTAs that finish last (tried: 30 % slower).
    unsigned int nruns = 0, run_task = kPubEnd, since = 0;
    auto write_stat = [&](const PsTaskDev* T, double tot) {
      PsStat stt;
      stt.sqnorm = tot;
      stt.step = T->step;
      stt.busy_ns = 0; stt.t_first = 0; stt.t_last = 0; stt._r0 = 0;
      stats[T->stat_idx] = stt;
    };
    auto flush = [&]() {
      __syncwarp();
      if (nruns == 0) return;
      __threadfence();                                  // this warp's partial sums before its tickets
      const unsigned int i = lane;                      // (kPubRuns <= 32: one lane per run)
      const bool have = i < nruns;
      const unsigned int t = have ? s_run_task[i] : 0u;
      const unsigned int add = have ? s_run_chunks[i] : 0u;
      bool last = false;
      if (have) last = atomicAdd(&tasks[t].ticket, add) + add == tasks[t].nchunks;
      unsigned int todo = __ballot_sync(0xffffffffu, last);
      if (todo) __threadfence();                        // the other CTAs' partial sums after the ticket
      while (todo) {
        const int src = __ffs(todo) - 1;
        todo &= todo - 1;
        const PsTaskDev* T = tasks + __shfl_sync(0xffffffffu, t, src);
        const double tot = sum_partials_warp(partials + T->first_chunk, T->nchunks, lane);
        if (lane == 0) write_stat(T, tot);
      }
      nruns = 0;
      run_task = kPubEnd;
      __syncwarp();
    };
    for (unsigned int k = 0;; ++k) {
      const unsigned int slot = k % (unsigned int)kPubSlots, parity = (k / (unsigned int)kPubSlots) & 1u;
      if (!__all_sync(0xffffffffu, mbar_wait(&pub_bar[slot], parity, &s_abort, wait_limit))) {
        if (lane == 0) {
          s_abort = 1;
          atomicExch(status, 3);
        }
        break;
      }
      const unsigned int t = s_pub_task[slot], c = s_pub_chunk[slot];
      if (t == kPubEnd) {
        flush();
        break;
      }
      // the chunk's sum of squares: its eight shares added in warp order
      double sum = 0.0;
      if (lane == 0) {
#pragma unroll
        for (int w = 0; w < kBulkConsumerWarps; ++w) sum += s_part[slot][w];
      }
      const PsTaskDev* T = tasks + t;
      if (T->nchunks == 1) {                            // nobody else to wait for: no ticket, no fence
        if (lane == 0) write_stat(T, sum);
      } else {
        if (lane == 0) __stcg(partials + c, sum);
        if (since == (unsigned int)kPubRuns) {
          flush();
          since = 0;
        }
        ++since;
        if (t != run_task) {                            // consecutive chunks of one task share a ticket draw
          if (lane == 0) {
            s_run_task[nruns] = t;
            s_run_chunks[nruns] = 0;
          }
          run_task = t;
          ++nruns;
        }
        __syncwarp();
        if (lane == 0) ++s_run_chunks[nruns - 1];
      }
      __syncwarp();
      if (lane == 0) *const_cast<volatile unsigned int*>(&s_pub_done) = k + 1;    // the slot may be filled again
    }
  } else {
    // -------------------------------------------------------------- consumer warps
    unsigned int stage = 0, takes = 0;
    double sq = 0.0;
    float acc[16];
#pragma unroll
    for (int k = 0; k < 16; ++k) acc[k] = 0.f;
    while (true) {
      // all lanes poll; the outcome is made warp-uniform before anyone leaves
      if (!__all_sync(0xffffffffu, mbar_wait(&full_bar[stage], (takes / kStages) & 1u, &s_abort, wait_limit))) {
        if (lane == 0) {
          s_abort = 1;
          atomicExch(status, 2);
        }
        break;
      }
      const StageMeta& m = meta[stage];
      const unsigned int flags = m.flags;
      if (flags & kTileEnd) break;
      const unsigned char* st = ring + (size_t)stage * kStageBytes;
      const unsigned int task = m.task, chunk = m.chunk;
      if (flags & kTileDirect) {
        const PsTaskDev* T = tasks + task;
        const unsigned int chunk_elems = T->chunk_elems;
        const size_t begin = (size_t)(chunk - T->first_chunk) * chunk_elems;
        const unsigned int count = (unsigned int)min((unsigned long long)chunk_elems, T->nelem - begin);
        run_chunk_any<kBulkConsumers>(tid, jobs + T->job, T, ptrs + T->shard_row, begin, count, sq);
      } else {
        const bool first = (flags & kTileFirst) != 0;
        if (m.kind & 1) ring_accumulate<true>(tid, st, m.nrows, m.cnt, first, acc);
        else ring_accumulate<false>(tid, st, m.nrows, m.cnt, first, acc);
        if (flags & kTileLast) {
          switch (m.kind) {
            case 0: ring_update<0, false>(tid, m, st, acc, sq); break;
            case 1: ring_update<0, true>(tid, m, st, acc, sq); break;
            case 2: ring_update<1, false>(tid, m, st, acc, sq); break;
            default: ring_update<1, true>(tid, m, st, acc, sq); break;
          }
          if (flags & kChunkEnd) {
            // the chunk's last few elements (fewer than one vector) bypass the ring
            const PsTaskDev* T = tasks + task;
            const unsigned int chunk_elems = T->chunk_elems;
            const size_t begin = (size_t)(chunk - T->first_chunk) * chunk_elems;
            const unsigned int count = (unsigned int)min((unsigned long long)chunk_elems, T->nelem - begin);
            const unsigned int vecw = (m.kind & 1) ? 8u : 4u;
            const unsigned int body = count & ~(vecw - 1);
            if (body != count) {
              const void* const* shards = ptrs + T->shard_row;
              switch (m.kind) {
                case 0: chunk_scalar<0, false, kBulkConsumers>(tid, m.h, shards, m.W, m.p, m.s0, m.s1, begin, body, count, sq); break;
                case 1: chunk_scalar<0, true, kBulkConsumers>(tid, m.h, shards, m.W, m.p, m.s0, m.s1, begin, body, count, sq); break;
                case 2: chunk_scalar<1, false, kBulkConsumers>(tid, m.h, shards, m.W, m.p, m.s0, m.s1, begin, body, count, sq); break;
                default: chunk_scalar<1, true, kBulkConsumers>(tid, m.h, shards, m.W, m.p, m.s0, m.s1, begin, body, count, sq); break;
              }
            }
          }
        }
      }
      if (flags & kChunkEnd) {
        // this warp's share of the chunk's sum of squares, left for the publisher warp
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sq += __shfl_down_sync(0xffffffffu, sq, o);
        if (lane == 0) {
          s_part[m.pub_slot][warp] = sq;
          mbar_arrive(&pub_bar[m.pub_slot]);
        }
        sq = 0.0;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty_bar[stage]);     // this warp is done with the stage
      ++takes;
      stage = (stage + 1 == kStages) ? 0 : stage + 1;
    }
  }
  signal_exit(&hdr->exited, done_word, seq);
}

}  // namespace psb
