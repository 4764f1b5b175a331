// Chunk body for tasks whose workers pushed ROW-SPARSE shards (embedding
// tables): a worker sends only the rows it touched, as a sorted list of row ids
// plus the packed rows.  The result is the dense one with the missing rows read
// as +0.0 — the aggregate is still the sum over workers 0..W-1 in that order —
// but only the rows that exist are read.
//
// One warp owns a row at a time.  Lane w looks worker w's shard up (a cursor
// over its sorted ids that only moves forward inside a chunk), the warp votes
// which workers hold the row, the sources are compacted in worker order into
// shared memory, and then all lanes stream the row: sum the present shards in
// order, apply the optimizer, store.
//
// Signed zero: adding an absent worker's +0.0 changes a running sum only when
// that sum is -0.0, and once it is +0.0 further -0.0 terms keep it +0.0; so the
// dense result equals the sum of the present shards, plus one "+ 0.0f" when at
// least one worker is absent.
#pragma once

#include "ps_math.cuh"

namespace psb {

constexpr int kRowsMaxWorkers = 32;   // one lane per worker

__device__ __forceinline__ unsigned int lower_bound_ids(const int* ids, unsigned int n, int key) {
  unsigned int lo = 0, hi = n;
  while (lo < hi) {
    const unsigned int mid = (lo + hi) >> 1;
    if (__ldg(ids + mid) < key) lo = mid + 1; else hi = mid;
  }
  return lo;
}

// srcs: this warp's 32 slots of shared memory.
template <int OPT, bool BF16, int NT>
__device__ __forceinline__ void chunk_rows(unsigned int tid, const Hp& h, const void* const* __restrict__ shards,
                                           const PsSparseDev* __restrict__ sparse, int W, float* __restrict__ p,
                                           float* __restrict__ s0, float* __restrict__ s1, size_t begin,
                                           unsigned int count, unsigned int row_len, const void** srcs, double& sq) {
  constexpr unsigned int V = BF16 ? 8 : 4;
  constexpr unsigned int ES = BF16 ? 2 : 4;
  const unsigned int lane = tid & 31, warp = tid >> 5;
  const unsigned int row0 = (unsigned int)(begin / row_len), nrows = count / row_len, groups = row_len / V;
  const bool mine = lane < (unsigned int)W;
  const int* ids = nullptr;
  unsigned int n = 0, cur = 0;
  const unsigned char* base = nullptr;
  if (mine) {
    base = static_cast<const unsigned char*>(ld_ptr(shards, lane));
    ids = sparse[lane].ids;
    n = sparse[lane].n;
    if (ids) cur = lower_bound_ids(ids, n, (int)(row0 + warp));
  }
  for (unsigned int r = row0 + warp; r < row0 + nrows; r += NT / 32) {
    bool present = false;
    const unsigned char* src = nullptr;
    if (mine) {
      if (!ids) {
        present = true;
        src = base + (size_t)r * row_len * ES;
      } else {
        while (cur < n && __ldg(ids + cur) < (int)r) ++cur;
        present = cur < n && __ldg(ids + cur) == (int)r;
        src = base + (size_t)cur * row_len * ES;
      }
    }
    const unsigned int mask = __ballot_sync(0xffffffffu, present);
    const unsigned int npresent = __popc(mask);
    const bool absent = npresent < (unsigned int)W;
    __syncwarp();                                            // the previous row's readers are done with srcs
    if (present) srcs[__popc(mask & ((1u << lane) - 1u))] = src;
    __syncwarp();
    const size_t e_row = (size_t)r * row_len;
    for (unsigned int g = lane; g < groups; g += 32) {
      const size_t e = e_row + (size_t)g * V;
      if (!BF16) {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        if (npresent) acc = as_f4(ld_stream(static_cast<const unsigned char*>(srcs[0]) + (size_t)g * 16));
#pragma unroll 4
        for (unsigned int k = 1; k < npresent; ++k)
          acc = add4(acc, ld_stream(static_cast<const unsigned char*>(srcs[k]) + (size_t)g * 16));
        if (absent) {
          acc.x = __fadd_rn(acc.x, 0.f); acc.y = __fadd_rn(acc.y, 0.f);
          acc.z = __fadd_rn(acc.z, 0.f); acc.w = __fadd_rn(acc.w, 0.f);
        }
        const float4 pv = *reinterpret_cast<const float4*>(p + e);
        const float4 av = *reinterpret_cast<const float4*>(s0 + e);
        const float4 bv = (OPT == 1) ? *reinterpret_cast<const float4*>(s1 + e) : make_float4(0, 0, 0, 0);
        update4<OPT>(h, acc, p, s0, s1, e, pv, av, bv, sq);
      } else {
        float acc[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) acc[q] = 0.f;
        if (npresent) widen8(ld_stream(static_cast<const unsigned char*>(srcs[0]) + (size_t)g * 16), acc);
#pragma unroll 4
        for (unsigned int k = 1; k < npresent; ++k) {
          float v[8];
          widen8(ld_stream(static_cast<const unsigned char*>(srcs[k]) + (size_t)g * 16), v);
#pragma unroll
          for (int q = 0; q < 8; ++q) acc[q] = __fadd_rn(acc[q], v[q]);
        }
        if (absent) {
#pragma unroll
          for (int q = 0; q < 8; ++q) acc[q] = __fadd_rn(acc[q], 0.f);
        }
        const float4 z = make_float4(0, 0, 0, 0);
        const float4 p0 = *reinterpret_cast<const float4*>(p + e), p1 = *reinterpret_cast<const float4*>(p + e + 4);
        const float4 a0 = *reinterpret_cast<const float4*>(s0 + e), a1 = *reinterpret_cast<const float4*>(s0 + e + 4);
        const float4 b0 = (OPT == 1) ? *reinterpret_cast<const float4*>(s1 + e) : z;
        const float4 b1 = (OPT == 1) ? *reinterpret_cast<const float4*>(s1 + e + 4) : z;
        update4<OPT>(h, make_float4(acc[0], acc[1], acc[2], acc[3]), p, s0, s1, e, p0, a0, b0, sq);
        update4<OPT>(h, make_float4(acc[4], acc[5], acc[6], acc[7]), p, s0, s1, e + 4, p1, a1, b1, sq);
      }
    }
  }
}

template <int NT>
__device__ __forceinline__ void run_rows_any(unsigned int tid, const PsJobDev* J, const PsTaskDev* T,
                                             const void* const* shards, const PsSparseDev* sparse, size_t begin,
                                             unsigned int count, const void** srcs, double& sq) {
  const Hp h = load_hp(J, T);
  const int W = J->W;
  const unsigned int rl = T->row_len;
  switch ((J->opt << 1) | J->grad_dtype) {
    case 0: chunk_rows<0, false, NT>(tid, h, shards, sparse, W, T->p, T->s0, T->s1, begin, count, rl, srcs, sq); break;
    case 1: chunk_rows<0, true, NT>(tid, h, shards, sparse, W, T->p, T->s0, T->s1, begin, count, rl, srcs, sq); break;
    case 2: chunk_rows<1, false, NT>(tid, h, shards, sparse, W, T->p, T->s0, T->s1, begin, count, rl, srcs, sq); break;
    default: chunk_rows<1, true, NT>(tid, h, shards, sparse, W, T->p, T->s0, T->s1, begin, count, rl, srcs, sq); break;
  }
}

}  // namespace psb
