// Aggregation kernel, bulk-copy variant for sm_100a: one persistent CTA per SM,
// warp-specialised.  A producer warp claims (job, block, chunk) work items from
// the table's atomic counter, cuts each chunk into tiles and streams every
// tile's rows — the W gradient shards, the parameters and the optimizer state —
// into a shared-memory ring with 1-D bulk asynchronous copies (TMA unit,
// completion counted on an mbarrier; every CTA fetches its own tiles).  Eight consumer
// warps take tiles out of the ring, sum the shards in worker order 0..W-1 in
// binary32, apply the optimizer and store parameters and state back with
// 128-bit stores.  The ring keeps several tiles (about 160 KB per SM) in flight
// independent of W, which direct loads cannot do for jobs with few workers.
//
// Chunks that cannot use bulk copies (a shard pointer that is not 16-byte
// aligned, or so many workers that a 128-element tile does not fit a stage) are
// handed to the consumers as "direct" work and read with ordinary loads.
// Warps synchronise through mbarriers only (never a CTA-wide barrier after the
// set-up), and every mbarrier wait is bounded: on expiry the warp records an
// error code in the device status word and leaves; the producer first lets its
// own copies land.
#pragma once

#include "ps_math.cuh"

namespace psb {

constexpr int kBulkConsumerWarps = 8;
constexpr int kBulkConsumers = kBulkConsumerWarps * 32;     // 256 consumer threads
constexpr int kBulkThreads = kBulkConsumers + 32;           // + one producer warp
constexpr int kStageBytes = 32768;
constexpr int kStages = 6;
constexpr int kBulkSmemBytes = kStages * kStageBytes + 1024;
constexpr unsigned int kTileQuantum = 128;                  // tile_elems is a multiple of this
constexpr long long kWaitCycles = 4000000000ll;             // about 2 s at 2 GHz

enum : unsigned int { kTileFirst = 1u, kTileLast = 2u, kTileDirect = 4u, kTileEnd = 8u };

struct TileMeta {
  unsigned int task, chunk, off, cnt, flags;   // off/cnt: vector-body elements inside the chunk
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
// Bounded wait.  Returns false if the limit expired or another warp aborted.
__device__ __forceinline__ bool mbar_wait(unsigned long long* bar, unsigned int parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  unsigned int spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 255u) == 0) {
      if (*abort_flag) return false;
      if (clock64() - t0 > kWaitCycles) return false;
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

// ---- consumer tile bodies ----------------------------------------------------

// fp32 shards: rows of `T` floats; row w < W = shard w, then p, s0, (s1).
template <int OPT>
__device__ __forceinline__ void tile_f32(unsigned int c, const Hp& h, const float* __restrict__ sm, int W,
                                         unsigned int T, unsigned int cnt, float* __restrict__ p,
                                         float* __restrict__ s0, float* __restrict__ s1, size_t e0, double& sq) {
  const unsigned int nvec = cnt >> 2;
  const float4* rp = reinterpret_cast<const float4*>(sm + (size_t)W * T);
  const float4* ra = reinterpret_cast<const float4*>(sm + (size_t)(W + 1) * T);
  const float4* rb = reinterpret_cast<const float4*>(sm + (size_t)(W + 2) * T);
  for (unsigned int g = c; g < nvec; g += kBulkConsumers) {
    float4 acc = reinterpret_cast<const float4*>(sm)[g];
#pragma unroll 8
    for (int w = 1; w < W; ++w) acc = add4(acc, reinterpret_cast<const uint4*>(sm + (size_t)w * T)[g]);
    const float4 bv = (OPT == 1) ? rb[g] : make_float4(0, 0, 0, 0);
    update4<OPT>(h, acc, p, s0, s1, e0 + 4 * (size_t)g, rp[g], ra[g], bv, sq);
  }
}

// bf16 shards: rows of `T` bf16 (2T bytes); then fp32 rows p, s0, (s1).
template <int OPT>
__device__ __forceinline__ void tile_bf16(unsigned int c, const Hp& h, const unsigned char* __restrict__ sm, int W,
                                          unsigned int T, unsigned int cnt, float* __restrict__ p,
                                          float* __restrict__ s0, float* __restrict__ s1, size_t e0, double& sq) {
  const unsigned int nvec = cnt >> 3;
  const float4* rp = reinterpret_cast<const float4*>(sm + (size_t)W * T * 2);
  const float4* ra = rp + T / 4;
  const float4* rb = ra + T / 4;
  for (unsigned int g = c; g < nvec; g += kBulkConsumers) {
    float acc[8];
    widen8(reinterpret_cast<const uint4*>(sm)[g], acc);
#pragma unroll 8
    for (int w = 1; w < W; ++w) {
      float v[8];
      widen8(reinterpret_cast<const uint4*>(sm + (size_t)w * T * 2)[g], v);
#pragma unroll
      for (int k = 0; k < 8; ++k) acc[k] = __fadd_rn(acc[k], v[k]);
    }
    const float4 z = make_float4(0, 0, 0, 0);
    const size_t e = e0 + 8 * (size_t)g;
    update4<OPT>(h, make_float4(acc[0], acc[1], acc[2], acc[3]), p, s0, s1, e, rp[2 * g], ra[2 * g],
                 (OPT == 1) ? rb[2 * g] : z, sq);
    update4<OPT>(h, make_float4(acc[4], acc[5], acc[6], acc[7]), p, s0, s1, e + 4, rp[2 * g + 1], ra[2 * g + 1],
                 (OPT == 1) ? rb[2 * g + 1] : z, sq);
  }
}

// ---- the kernel ----------------------------------------------------------------

__global__ void __launch_bounds__(kBulkThreads, 1)
ps_aggregate_bulk_kernel(unsigned char* __restrict__ table, const PsJobDev* __restrict__ jobs,
                         PsStat* __restrict__ stats, double* __restrict__ partials, int* __restrict__ status) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* ring = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127);
  __shared__ __align__(8) unsigned long long full_bar[kStages];
  __shared__ __align__(8) unsigned long long empty_bar[kStages];
  __shared__ TileMeta meta[kStages];
  __shared__ int s_abort;

  PsTableHdr* hdr = reinterpret_cast<PsTableHdr*>(table);
  PsTaskDev* tasks = reinterpret_cast<PsTaskDev*>(table + hdr->tasks_off);
  const unsigned int* starts = reinterpret_cast<const unsigned int*>(table + hdr->starts_off);
  const void* const* ptrs = reinterpret_cast<const void* const*>(table + hdr->ptrs_off);
  const unsigned int n_tasks = hdr->n_tasks, total = hdr->total_chunks;

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
    unsigned int cursor = 0, stage = 0, fills = 0;   // fills: tiles posted so far
    unsigned int pend_mask = 0, pend_par = 0;        // stages whose last fill carried copies, and its parity
    bool ok = true;
    unsigned int idx = 0, next = 0;
    if (lane == 0) idx = atomicAdd(&hdr->counter, 1u);
    idx = __shfl_sync(0xffffffffu, idx, 0);
    while (ok && idx < total) {
      if (lane == 0) next = atomicAdd(&hdr->counter, 1u);      // overlaps this chunk's copies
      cursor = find_task(starts, n_tasks, cursor, idx, lane);
      const PsTaskDev* T = tasks + cursor;
      const PsJobDev* J = jobs + T->job;
      const int W = J->W;
      const unsigned int ges = J->grad_dtype ? 2u : 4u;
      const unsigned int vecw = J->grad_dtype ? 8u : 4u;
      const int nstate = J->opt ? 2 : 1;
      const unsigned int chunk_elems = T->chunk_elems;
      const size_t begin = (size_t)(idx - T->first_chunk) * chunk_elems;
      const unsigned int count = (unsigned int)min((unsigned long long)chunk_elems, T->nelem - begin);
      const unsigned int tile = T->tile_elems;
      const bool direct = tile == 0 || T->vec_ok == 0;
      const unsigned int body = direct ? 0u : (count & ~(vecw - 1));
      const unsigned int ntiles = direct ? 1u : max(1u, (body + tile - 1) / tile);
      const void* const* shards = ptrs + T->shard_row;
      for (unsigned int k = 0; k < ntiles; ++k) {
        const unsigned int use = fills / kStages;
        if (use > 0) ok = mbar_wait(&empty_bar[stage], (use - 1) & 1u, &s_abort);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        const unsigned int off = k * tile;
        const unsigned int cnt = direct ? 0u : min(tile, body - off);
        unsigned char* dst = ring + (size_t)stage * kStageBytes;
        if (lane == 0) {
          TileMeta m;
          m.task = cursor; m.chunk = idx; m.off = off; m.cnt = cnt;
          m.flags = (k == 0 ? kTileFirst : 0u) | (k == ntiles - 1 ? kTileLast : 0u) | (direct ? kTileDirect : 0u);
          meta[stage] = m;
          if (cnt) mbar_arrive_expect_tx(&full_bar[stage], cnt * ((unsigned int)W * ges + 4u * (1 + nstate)));
          else mbar_arrive(&full_bar[stage]);
        }
        __syncwarp();
        if (cnt) {
          const size_t e = begin + off;
          const unsigned int rows = (unsigned int)W + 1 + nstate;
          for (unsigned int r = lane; r < rows; r += 32) {
            if (r < (unsigned int)W) {
              const unsigned char* src = static_cast<const unsigned char*>(ld_ptr(shards, r)) + e * ges;
              bulk_g2s(dst + (size_t)r * tile * ges, src, cnt * ges, &full_bar[stage]);
            } else {
              const unsigned int q = r - W;
              const float* src = (q == 0 ? T->p : (q == 1 ? T->s0 : T->s1)) + e;
              bulk_g2s(dst + (size_t)W * tile * ges + (size_t)q * tile * 4, src, cnt * 4, &full_bar[stage]);
            }
          }
          pend_mask |= 1u << stage;
          pend_par = (pend_par & ~(1u << stage)) | ((use & 1u) << stage);
        } else {
          pend_mask &= ~(1u << stage);
        }
        ++fills;
        stage = (stage + 1 == kStages) ? 0 : stage + 1;
      }
      idx = __shfl_sync(0xffffffffu, next, 0);
    }
    // end marker for the consumers
    if (ok) {
      const unsigned int use = fills / kStages;
      if (use > 0) ok = mbar_wait(&empty_bar[stage], (use - 1) & 1u, &s_abort);
      ok = __all_sync(0xffffffffu, ok);
      if (ok && lane == 0) {
        TileMeta m;
        m.task = 0; m.chunk = 0; m.off = 0; m.cnt = 0; m.flags = kTileEnd;
        meta[stage] = m;
        mbar_arrive(&full_bar[stage]);
      }
    }
    if (!ok) {
      // expired wait: flag it, then let this CTA's own copies land before leaving
      if (lane == 0) {
        s_abort = 1;
        atomicExch(status, 1);
        for (int s = 0; s < kStages; ++s)
          if ((pend_mask >> s) & 1u) {
            const long long t0 = clock64();
            while (!mbar_try_wait(&full_bar[s], (pend_par >> s) & 1u) && clock64() - t0 < kWaitCycles) {}
          }
      }
      __syncwarp();
    }
    return;
  }

  // -------------------------------------------------------------- consumer warps
  unsigned int stage = 0, takes = 0;
  double sq = 0.0;
  unsigned int cur_task = 0xffffffffu;
  Hp h;
  int W = 0, kind = 0;
  float *p = nullptr, *s0 = nullptr, *s1 = nullptr;
  while (true) {
    // all lanes poll; the outcome is made warp-uniform before anyone leaves
    if (!__all_sync(0xffffffffu, mbar_wait(&full_bar[stage], (takes / kStages) & 1u, &s_abort))) {
      if (lane == 0) {
        s_abort = 1;
        atomicExch(status, 2);
      }
      return;
    }
    const TileMeta m = meta[stage];
    if (m.flags & kTileEnd) break;
    const PsTaskDev* T = tasks + m.task;
    const PsJobDev* J = jobs + T->job;
    if (m.task != cur_task) {
      cur_task = m.task;
      h = load_hp(J, T);
      W = J->W;
      kind = (J->opt << 1) | J->grad_dtype;
      p = T->p; s0 = T->s0; s1 = T->s1;
    }
    const unsigned int chunk_elems = T->chunk_elems;
    const size_t begin = (size_t)(m.chunk - T->first_chunk) * chunk_elems;
    const unsigned int count = (unsigned int)min((unsigned long long)chunk_elems, T->nelem - begin);
    if (m.flags & kTileDirect) {
      run_chunk_any<kBulkConsumers>(tid, J, T, ptrs + T->shard_row, begin, count, sq);
    } else {
      const unsigned char* sm = ring + (size_t)stage * kStageBytes;
      const unsigned int tile = T->tile_elems;
      const size_t e0 = begin + m.off;
      switch (kind) {
        case 0: tile_f32<0>(tid, h, reinterpret_cast<const float*>(sm), W, tile, m.cnt, p, s0, s1, e0, sq); break;
        case 1: tile_bf16<0>(tid, h, sm, W, tile, m.cnt, p, s0, s1, e0, sq); break;
        case 2: tile_f32<1>(tid, h, reinterpret_cast<const float*>(sm), W, tile, m.cnt, p, s0, s1, e0, sq); break;
        default: tile_bf16<1>(tid, h, sm, W, tile, m.cnt, p, s0, s1, e0, sq); break;
      }
      if (m.flags & kTileLast) {
        // the chunk's last few elements (fewer than one vector) bypass the ring
        const unsigned int vecw = (kind & 1) ? 8u : 4u;
        const unsigned int body = count & ~(vecw - 1);
        if (body != count) {
          const void* const* shards = ptrs + T->shard_row;
          switch (kind) {
            case 0: chunk_scalar<0, false, kBulkConsumers>(tid, h, shards, W, p, s0, s1, begin, body, count, sq); break;
            case 1: chunk_scalar<0, true, kBulkConsumers>(tid, h, shards, W, p, s0, s1, begin, body, count, sq); break;
            case 2: chunk_scalar<1, false, kBulkConsumers>(tid, h, shards, W, p, s0, s1, begin, body, count, sq); break;
            default: chunk_scalar<1, true, kBulkConsumers>(tid, h, shards, W, p, s0, s1, begin, body, count, sq); break;
          }
        }
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&empty_bar[stage]);     // this warp is done reading the stage
    ++takes;
    stage = (stage + 1 == kStages) ? 0 : stage + 1;

    if (m.flags & kTileLast) {
      // this warp's share of the chunk's sum of squares; the warps never meet
      // at a CTA barrier, each publishes its own partial
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sq += __shfl_down_sync(0xffffffffu, sq, o);
      publish_part(tasks, m.task, m.chunk * kBulkConsumerWarps + warp, kBulkConsumerWarps, sq, stats, partials, lane);
      sq = 0.0;
    }
  }
}

}  // namespace psb
