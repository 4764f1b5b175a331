// Aggregation kernel, bulk-copy variant for sm_100a: one persistent CTA per SM,
// warp-specialised.  A producer warp claims (job, block, chunk) work items from
// the table's atomic counter, cuts each chunk into tiles of 2048 elements and
// streams every tile into a shared-memory ring with 1-D bulk asynchronous
// copies (TMA unit, completion counted on an mbarrier; every CTA fetches its own
// tiles, no multicast).  A tile is cut ALONG THE WORKERS: one ring stage holds
// the tile's rows of a few consecutive workers (four fp32 or eight bf16 shards,
// 8 KB or 4 KB per row, so every copy is large), the next stage the next
// workers, and the parameters and optimizer state ride in the tile's last
// stage.  Eight consumer warps keep the running sums of a tile in registers
// across its stages — worker order 0..W-1, binary32, so the bits are those of
// the direct-load kernel — and on the last stage apply the optimizer and store
// parameters and state with 128-bit stores.  The ring keeps 192 KB per SM in
// flight whatever W is.
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
constexpr int kBulkThreads = kBulkConsumers + 32;           // + one producer warp
constexpr int kStageBytes = 32768;
constexpr int kStages = 6;
constexpr int kBulkSmemBytes = kStages * kStageBytes + 1024;
constexpr unsigned int kRingTile = 2048;                    // elements per tile: 8 per consumer thread
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

// Adds the stage's shard rows to the thread's running sums.  fp32: the thread owns
// the float4 groups c and c + 256 of the tile; bf16: the 8 elements of group c.
template <bool BF16>
__device__ __forceinline__ void ring_accumulate(unsigned int c, const unsigned char* __restrict__ st, unsigned int nrows,
                                                unsigned int cnt, bool first, float (&acc)[8]) {
  if (!BF16) {
    const unsigned int ng = cnt >> 2;
    const bool a0 = c < ng, a1 = c + kBulkConsumers < ng;
    constexpr unsigned int kRow = kRingTile * 4;
#pragma unroll 4
    for (unsigned int r = 0; r < nrows; ++r) {
      const uint4* row = reinterpret_cast<const uint4*>(st + (size_t)r * kRow);
      uint4 x0 = make_uint4(0, 0, 0, 0), x1 = x0;
      if (a0) x0 = row[c];
      if (a1) x1 = row[c + kBulkConsumers];
      if (first && r == 0) {
        acc[0] = __uint_as_float(x0.x); acc[1] = __uint_as_float(x0.y); acc[2] = __uint_as_float(x0.z); acc[3] = __uint_as_float(x0.w);
        acc[4] = __uint_as_float(x1.x); acc[5] = __uint_as_float(x1.y); acc[6] = __uint_as_float(x1.z); acc[7] = __uint_as_float(x1.w);
      } else {
        acc[0] = __fadd_rn(acc[0], __uint_as_float(x0.x)); acc[1] = __fadd_rn(acc[1], __uint_as_float(x0.y));
        acc[2] = __fadd_rn(acc[2], __uint_as_float(x0.z)); acc[3] = __fadd_rn(acc[3], __uint_as_float(x0.w));
        acc[4] = __fadd_rn(acc[4], __uint_as_float(x1.x)); acc[5] = __fadd_rn(acc[5], __uint_as_float(x1.y));
        acc[6] = __fadd_rn(acc[6], __uint_as_float(x1.z)); acc[7] = __fadd_rn(acc[7], __uint_as_float(x1.w));
      }
    }
  } else {
    const unsigned int ng = cnt >> 3;
    const bool a0 = c < ng;
    constexpr unsigned int kRow = kRingTile * 2;
#pragma unroll 4
    for (unsigned int r = 0; r < nrows; ++r) {
      uint4 x = make_uint4(0, 0, 0, 0);
      if (a0) x = reinterpret_cast<const uint4*>(st + (size_t)r * kRow)[c];
      if (first && r == 0) {
        widen8(x, acc);
      } else {
        add_bf16x2(acc[0], acc[1], x.x);
        add_bf16x2(acc[2], acc[3], x.y);
        add_bf16x2(acc[4], acc[5], x.z);
        add_bf16x2(acc[6], acc[7], x.w);
      }
    }
  }
}

// The tile's last stage: parameters and state come out of the ring, the update goes to global memory.
template <int OPT, bool BF16>
__device__ __forceinline__ void ring_update(unsigned int c, const StageMeta& m, const unsigned char* __restrict__ st,
                                            const float (&acc)[8], double& sq) {
  const float4* rp = reinterpret_cast<const float4*>(st + m.state_off);
  const float4* ra = rp + kRingTile / 4;
  const float4* rb = ra + kRingTile / 4;
  const unsigned int ng4 = m.cnt >> 2;
  const float4 z = make_float4(0, 0, 0, 0);
  // fp32: groups c and c + 256; bf16: groups 2c and 2c + 1 (the thread's 8 consecutive elements)
  const unsigned int g0 = BF16 ? 2 * c : c, g1 = BF16 ? 2 * c + 1 : c + kBulkConsumers;
  if (g0 < ng4)
    update4<OPT>(m.h, make_float4(acc[0], acc[1], acc[2], acc[3]), m.p, m.s0, m.s1, (size_t)m.e0 + 4 * (size_t)g0,
                 rp[g0], ra[g0], OPT == 1 ? rb[g0] : z, sq);
  if (g1 < ng4)
    update4<OPT>(m.h, make_float4(acc[4], acc[5], acc[6], acc[7]), m.p, m.s0, m.s1, (size_t)m.e0 + 4 * (size_t)g1,
                 rp[g1], ra[g1], OPT == 1 ? rb[g1] : z, sq);
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
  __shared__ double s_part[kStages][kBulkConsumerWarps];   // a chunk's sums of squares, one per consumer warp
  __shared__ unsigned int s_pub_task[kStages], s_pub_chunk[kStages];
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
    s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();

  if (warp == kBulkConsumerWarps) {
    // ------------------------------------------------------------ producer warp
    unsigned int cursor = 0, stage = 0, fills = 0;   // fills: stages posted so far
    unsigned int pend_mask = 0, pend_par = 0;        // stages whose last fill carried copies, and its parity
    unsigned int pub_mask = 0, pub_par = 0;          // stages that closed a chunk whose partial sums are not published yet
    bool ok = true;
    unsigned int idx = 0, next = 0;
    if (lane == 0) idx = atomicAdd(&hdr->counter, 1u);
    idx = __shfl_sync(0xffffffffu, idx, 0);

    // Posts one stage: waits for the slot, publishes its description, arms the barrier and
    // issues the copies (lane l fetches row l of the stage).  nsh shard rows from worker
    // `first_w`, then nst state rows if this is the tile's last stage.
    // The consumers leave a finished chunk's eight partial sums of squares in shared memory
    // before they release the chunk's last stage; the producer publishes them when it next
    // owns that stage.  (Published by the consumers themselves, the fence before the ticket
    // made each of the eight warps wait for its own parameter stores once per chunk: the
    // largest stall of the kernel.  The producer has no stores of its own in flight.)
    auto publish = [&](unsigned int st) {
      const unsigned int t = s_pub_task[st], c = s_pub_chunk[st];
      const PsTaskDev* T = tasks + t;
      const unsigned int first = T->first_chunk * kBulkConsumerWarps, n = T->nchunks * kBulkConsumerWarps;
      if (lane < kBulkConsumerWarps) __stcg(partials + (size_t)c * kBulkConsumerWarps + lane, s_part[st][lane]);
      __syncwarp();
      unsigned int done = 0;
      if (lane == 0) {
        __threadfence();
        done = atomicAdd(&tasks[t].ticket, (unsigned int)kBulkConsumerWarps);
        __threadfence();
      }
      done = __shfl_sync(0xffffffffu, done, 0);
      if (done == n - kBulkConsumerWarps) {
        const double tot = sum_partials_warp(partials + first, n, lane);
        if (lane == 0) {
          PsStat stt;
          stt.sqnorm = tot;
          stt.step = T->step;
          stt.busy_ns = 0; stt.t_first = 0; stt.t_last = 0; stt._r0 = 0;
          stats[T->stat_idx] = stt;
        }
      }
      pub_mask &= ~(1u << st);
    };

    // what every stage of a chunk repeats, read from the table once per chunk
    struct ChunkCtx {
      Hp h;
      float *p, *s0, *s1;
      const void* const* shards;
      int W, kind;
      unsigned int ges, nstate_rows;
    } cc = {};

    auto post = [&](unsigned int task, unsigned int chunk, size_t e0,
                    unsigned int cnt, unsigned int first_w, unsigned int nsh, bool with_state, unsigned int flags) {
      const unsigned int use = fills / kStages;
      if (use > 0) ok = mbar_wait(&empty_bar[stage], (use - 1) & 1u, &s_abort, wait_limit);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) return;
      if ((pub_mask >> stage) & 1u) publish(stage);
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
        m.W = cc.W;
        m.kind = cc.kind;
        m.h = cc.h;
        if (flags & kChunkEnd) {
          s_pub_task[stage] = task;
          s_pub_chunk[stage] = chunk;
        }
        if (bytes) mbar_arrive_expect_tx(&full_bar[stage], bytes);
        else mbar_arrive(&full_bar[stage]);
      }
      if (flags & kChunkEnd) {
        pub_mask |= 1u << stage;
        pub_par = (pub_par & ~(1u << stage)) | ((use & 1u) << stage);
      }
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

    while (ok && idx < total) {
      if (lane == 0) next = atomicAdd(&hdr->counter, 1u);      // overlaps this chunk's copies
      cursor = find_task(starts, n_tasks, cursor, idx, lane);
      const PsTaskDev* T = tasks + cursor;
      const PsJobDev* J = jobs + T->job;
      const unsigned int W = (unsigned int)J->W;
      const unsigned int ges = J->grad_dtype ? 2u : 4u;
      const unsigned int vecw = J->grad_dtype ? 8u : 4u;
      const unsigned int state_bytes = (J->opt ? 3u : 2u) * kRingTile * 4u;
      const unsigned int rows_per_stage = kStageBytes / (kRingTile * ges);
      const unsigned int chunk_elems = T->chunk_elems;
      const size_t begin = (size_t)(idx - T->first_chunk) * chunk_elems;
      const unsigned int count = (unsigned int)min((unsigned long long)chunk_elems, T->nelem - begin);
      const unsigned int body = count & ~(vecw - 1);
      cc.h = load_hp(J, T);
      cc.p = T->p; cc.s0 = T->s0; cc.s1 = T->s1;
      cc.shards = ptrs + T->shard_row;
      cc.W = J->W;
      cc.kind = (J->opt << 1) | J->grad_dtype;
      cc.ges = ges;
      cc.nstate_rows = J->opt ? 3u : 2u;
      if (T->tile_elems == 0 || T->vec_ok == 0 || body == 0) {
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
          }
        }
      }
      idx = __shfl_sync(0xffffffffu, next, 0);
    }
    // end marker for the consumers
    if (ok) {
      const unsigned int use = fills / kStages;
      if (use > 0) ok = mbar_wait(&empty_bar[stage], (use - 1) & 1u, &s_abort, wait_limit);
      ok = __all_sync(0xffffffffu, ok);
      if (ok) {
        if ((pub_mask >> stage) & 1u) publish(stage);
        if (lane == 0) {
          meta[stage].flags = kTileEnd;
          mbar_arrive(&full_bar[stage]);
        }
        // the chunks that ended in the other stages: published once the consumers have released them
        for (unsigned int st = 0; ok && st < (unsigned int)kStages; ++st) {
          if (!((pub_mask >> st) & 1u)) continue;
          ok = __all_sync(0xffffffffu, mbar_wait(&empty_bar[st], (pub_par >> st) & 1u, &s_abort, wait_limit));
          if (ok) publish(st);
        }
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
  } else {
    // -------------------------------------------------------------- consumer warps
    unsigned int stage = 0, takes = 0;
    double sq = 0.0;
    float acc[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) acc[k] = 0.f;
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
        // this warp's share of the chunk's sum of squares, left for the producer to publish
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sq += __shfl_down_sync(0xffffffffu, sq, o);
        if (lane == 0) s_part[stage][warp] = sq;
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
