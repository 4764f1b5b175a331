// Device-side data structures and kernels of the packed aggregation service.
//
// One launch serves any mix of jobs: the host uploads a task table — a header,
// one PsTaskDev per ready (job, block), the first chunk index of every task and
// the W shard pointers of every task — and persistent CTAs claim
// (job, block, chunk) work items from an atomic counter until the table is
// exhausted (paper Section 3.3: aggregation tasks of many jobs are packed onto
// one shared Aggregator; Section 2.2: tensors are independent, so chunks can be
// processed in any order by any CTA).
//
// Per chunk: the W gradient shards are read once with 128-bit loads, summed in
// binary32 in worker order 0..W-1 and fused with the optimizer update of the
// master copy and its state, so every byte crosses HBM once.  Explicit
// round-to-nearest intrinsics keep the compiler from fusing multiply-adds: the
// result is defined operation by operation in include/ps_b200.h.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace psb {

constexpr int kThreads = 256;          // threads per CTA
constexpr int kMaxWorkers = 256;

struct __align__(16) PsJobDev {        // 64 bytes, one per registered job
  int opt, grad_dtype, W, _pad;
  float lr, mom, wd, b1, b2, omb1, omb2, eps, gs, _r0, _r1, _r2;
};

struct __align__(16) PsTaskDev {       // 80 bytes, one per ready (job, block)
  float* p;
  float* s0;
  float* s1;
  unsigned long long nelem;
  unsigned int shard_row;              // index of the task's first shard pointer
  unsigned int first_chunk;
  unsigned int nchunks;
  unsigned int ticket;                 // chunks finished so far (uploaded as 0)
  float ss_t, sbc2_t;                  // Adam step size and sqrt(1 - b2^t)
  int job;
  unsigned int stat_idx;
  unsigned long long step;
  unsigned int vec_ok;                 // all pointers 16-byte aligned
  unsigned int _pad;
};

struct __align__(16) PsTableHdr {      // 32 bytes at the start of the table
  unsigned int counter;                // next chunk to claim (uploaded as 0)
  unsigned int n_tasks;
  unsigned int total_chunks;
  unsigned int chunk_elems;
  unsigned int tasks_off, starts_off, ptrs_off, _r0;   // byte offsets from the table base
};

struct __align__(16) PsStat {
  double sqnorm;
  unsigned long long step;
};

// ---------------------------------------------------------------- arithmetic

struct Hp {
  float lr, mom, wd, b1, b2, omb1, omb2, eps, gs, ss_t, sbc2_t;
};

template <int OPT>
__device__ __forceinline__ void update_elem(const Hp& h, float G, float& p, float& s0, float& s1, double& sq) {
  G = __fmul_rn(G, h.gs);
  sq = fma((double)G, (double)G, sq);      // binary64: product exact, sum rounded once
  const float d = __fadd_rn(G, __fmul_rn(h.wd, p));
  if (OPT == 0) {
    const float v = __fadd_rn(__fmul_rn(h.mom, s0), d);
    s0 = v;
    p = __fsub_rn(p, __fmul_rn(h.lr, v));
  } else {
    const float m = __fadd_rn(__fmul_rn(h.b1, s0), __fmul_rn(h.omb1, d));
    const float v = __fadd_rn(__fmul_rn(h.b2, s1), __fmul_rn(h.omb2, __fmul_rn(d, d)));
    const float den = __fadd_rn(__fdiv_rn(__fsqrt_rn(v), h.sbc2_t), h.eps);
    s0 = m;
    s1 = v;
    p = __fsub_rn(p, __fmul_rn(h.ss_t, __fdiv_rn(m, den)));
  }
}

__device__ __forceinline__ float bf16_lo(unsigned int u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(unsigned int u) { return __uint_as_float(u & 0xffff0000u); }

// Shard pointer w of a task, through the read-only path (uniform across the CTA).
__device__ __forceinline__ const void* ld_ptr(const void* const* shards, int w = 0) {
  return reinterpret_cast<const void*>(__ldg(reinterpret_cast<const unsigned long long*>(shards) + w));
}

// Streaming (read-once) 128-bit load.
__device__ __forceinline__ uint4 ld_stream(const void* p) { return __ldcs(reinterpret_cast<const uint4*>(p)); }

__device__ __forceinline__ float4 add4(float4 a, uint4 b) {
  a.x = __fadd_rn(a.x, __uint_as_float(b.x));
  a.y = __fadd_rn(a.y, __uint_as_float(b.y));
  a.z = __fadd_rn(a.z, __uint_as_float(b.z));
  a.w = __fadd_rn(a.w, __uint_as_float(b.w));
  return a;
}

template <int OPT>
__device__ __forceinline__ void update4(const Hp& h, const float4& G, float* p, float* s0, float* s1, size_t e,
                                        const float4& pv, const float4& av, const float4& bv, double& sq) {
  float4 P = pv, A = av, B = bv;
  update_elem<OPT>(h, G.x, P.x, A.x, B.x, sq);
  update_elem<OPT>(h, G.y, P.y, A.y, B.y, sq);
  update_elem<OPT>(h, G.z, P.z, A.z, B.z, sq);
  update_elem<OPT>(h, G.w, P.w, A.w, B.w, sq);
  *reinterpret_cast<float4*>(p + e) = P;
  *reinterpret_cast<float4*>(s0 + e) = A;
  if (OPT == 1) *reinterpret_cast<float4*>(s1 + e) = B;
}

// ---------------------------------------------------------------- chunk bodies

// fp32 gradients, 16-byte aligned: each thread owns U float4 groups per trip.
template <int OPT, int U>
__device__ __forceinline__ void chunk_f32_vec(const Hp& h, const void* const* __restrict__ shards, int W,
                                              float* __restrict__ p, float* __restrict__ s0, float* __restrict__ s1,
                                              size_t begin, unsigned int count, double& sq) {
  const unsigned int nvec = count >> 2;
  const unsigned int tid = threadIdx.x;
  unsigned int i = tid;
  // full trips: U groups per thread, no predicates
  for (; i + (U - 1) * kThreads < nvec; i += U * kThreads) {
    float4 acc[U], pv[U], av[U], bv[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const size_t e = begin + 4 * (size_t)(i + u * kThreads);
      pv[u] = *reinterpret_cast<const float4*>(p + e);
      av[u] = *reinterpret_cast<const float4*>(s0 + e);
      if (OPT == 1) bv[u] = *reinterpret_cast<const float4*>(s1 + e); else bv[u] = make_float4(0, 0, 0, 0);
    }
    {
      const float* g = static_cast<const float*>(ld_ptr(shards));
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const uint4 t = ld_stream(g + begin + 4 * (size_t)(i + u * kThreads));
        acc[u] = make_float4(__uint_as_float(t.x), __uint_as_float(t.y), __uint_as_float(t.z), __uint_as_float(t.w));
      }
    }
#pragma unroll 4
    for (int w = 1; w < W; ++w) {
      const float* g = static_cast<const float*>(ld_ptr(shards, w));
#pragma unroll
      for (int u = 0; u < U; ++u) acc[u] = add4(acc[u], ld_stream(g + begin + 4 * (size_t)(i + u * kThreads)));
    }
#pragma unroll
    for (int u = 0; u < U; ++u)
      update4<OPT>(h, acc[u], p, s0, s1, begin + 4 * (size_t)(i + u * kThreads), pv[u], av[u], bv[u], sq);
  }
  // remaining groups, one per thread
  for (; i < nvec; i += kThreads) {
    const size_t e = begin + 4 * (size_t)i;
    const float4 pv = *reinterpret_cast<const float4*>(p + e);
    const float4 av = *reinterpret_cast<const float4*>(s0 + e);
    const float4 bv = (OPT == 1) ? *reinterpret_cast<const float4*>(s1 + e) : make_float4(0, 0, 0, 0);
    const uint4 t = ld_stream(static_cast<const float*>(ld_ptr(shards)) + e);
    float4 acc = make_float4(__uint_as_float(t.x), __uint_as_float(t.y), __uint_as_float(t.z), __uint_as_float(t.w));
#pragma unroll 4
    for (int w = 1; w < W; ++w) acc = add4(acc, ld_stream(static_cast<const float*>(ld_ptr(shards, w)) + e));
    update4<OPT>(h, acc, p, s0, s1, e, pv, av, bv, sq);
  }
}

__device__ __forceinline__ void widen8(const uint4& t, float (&o)[8]) {
  o[0] = bf16_lo(t.x); o[1] = bf16_hi(t.x); o[2] = bf16_lo(t.y); o[3] = bf16_hi(t.y);
  o[4] = bf16_lo(t.z); o[5] = bf16_hi(t.z); o[6] = bf16_lo(t.w); o[7] = bf16_hi(t.w);
}

// bf16 gradients, 16-byte aligned: each thread owns 8 consecutive elements.
template <int OPT>
__device__ __forceinline__ void chunk_bf16_vec(const Hp& h, const void* const* __restrict__ shards, int W,
                                               float* __restrict__ p, float* __restrict__ s0, float* __restrict__ s1,
                                               size_t begin, unsigned int count, double& sq) {
  const unsigned int nvec = count >> 3;
  for (unsigned int i = threadIdx.x; i < nvec; i += kThreads) {
    const size_t e = begin + 8 * (size_t)i;
    const float4 p0 = *reinterpret_cast<const float4*>(p + e), p1 = *reinterpret_cast<const float4*>(p + e + 4);
    const float4 a0 = *reinterpret_cast<const float4*>(s0 + e), a1 = *reinterpret_cast<const float4*>(s0 + e + 4);
    float4 b0 = make_float4(0, 0, 0, 0), b1 = b0;
    if (OPT == 1) {
      b0 = *reinterpret_cast<const float4*>(s1 + e);
      b1 = *reinterpret_cast<const float4*>(s1 + e + 4);
    }
    float acc[8];
    widen8(ld_stream(static_cast<const unsigned short*>(ld_ptr(shards)) + e), acc);
#pragma unroll 8
    for (int w = 1; w < W; ++w) {
      float g[8];
      widen8(ld_stream(static_cast<const unsigned short*>(ld_ptr(shards, w)) + e), g);
#pragma unroll
      for (int k = 0; k < 8; ++k) acc[k] = __fadd_rn(acc[k], g[k]);
    }
    update4<OPT>(h, make_float4(acc[0], acc[1], acc[2], acc[3]), p, s0, s1, e, p0, a0, b0, sq);
    update4<OPT>(h, make_float4(acc[4], acc[5], acc[6], acc[7]), p, s0, s1, e + 4, p1, a1, b1, sq);
  }
}

// Any alignment, any count: one element per thread per trip.
template <int OPT, bool BF16>
__device__ __forceinline__ void chunk_scalar(const Hp& h, const void* const* __restrict__ shards, int W,
                                             float* __restrict__ p, float* __restrict__ s0, float* __restrict__ s1,
                                             size_t begin, unsigned int first, unsigned int count, double& sq) {
  for (unsigned int i = first + threadIdx.x; i < count; i += kThreads) {
    const size_t e = begin + i;
    float G;
    if (BF16) {
      G = __uint_as_float((unsigned int)__ldcs(static_cast<const unsigned short*>(ld_ptr(shards)) + e) << 16);
      for (int w = 1; w < W; ++w)
        G = __fadd_rn(G, __uint_as_float((unsigned int)__ldcs(static_cast<const unsigned short*>(ld_ptr(shards, w)) + e) << 16));
    } else {
      G = __ldcs(static_cast<const float*>(ld_ptr(shards)) + e);
      for (int w = 1; w < W; ++w) G = __fadd_rn(G, __ldcs(static_cast<const float*>(ld_ptr(shards, w)) + e));
    }
    float P = p[e], A = s0[e], B = (OPT == 1) ? s1[e] : 0.f;
    update_elem<OPT>(h, G, P, A, B, sq);
    p[e] = P;
    s0[e] = A;
    if (OPT == 1) s1[e] = B;
  }
}

template <int OPT, bool BF16>
__device__ __forceinline__ void run_chunk(const Hp& h, const void* const* shards, int W, float* p, float* s0, float* s1,
                                          size_t begin, unsigned int count, bool vec_ok, double& sq) {
  if (vec_ok) {
    constexpr unsigned int V = BF16 ? 8 : 4;
    const unsigned int body = count & ~(V - 1);
    if (BF16) chunk_bf16_vec<OPT>(h, shards, W, p, s0, s1, begin, body, sq);
    else chunk_f32_vec<OPT, 2>(h, shards, W, p, s0, s1, begin, body, sq);
    if (body != count) chunk_scalar<OPT, BF16>(h, shards, W, p, s0, s1, begin, body, count, sq);
  } else {
    chunk_scalar<OPT, BF16>(h, shards, W, p, s0, s1, begin, 0, count, sq);
  }
}

// ---------------------------------------------------------------- the kernel

// Persistent CTAs; each loop trip claims one chunk index from the table's
// counter (the next index is fetched while the current chunk is processed),
// finds its task by advancing a per-CTA cursor over the sorted first-chunk
// array, processes the chunk, and publishes the chunk's sum of squares.  The
// CTA that finishes a task's last chunk adds the task's partials in chunk
// order, so the per-block norm does not depend on which CTA ran which chunk.
__global__ void __launch_bounds__(kThreads, 3)
ps_aggregate_ldg_kernel(unsigned char* __restrict__ table, const PsJobDev* __restrict__ jobs,
                        PsStat* __restrict__ stats, double* __restrict__ partials) {
  PsTableHdr* hdr = reinterpret_cast<PsTableHdr*>(table);
  PsTaskDev* tasks = reinterpret_cast<PsTaskDev*>(table + hdr->tasks_off);
  const unsigned int* starts = reinterpret_cast<const unsigned int*>(table + hdr->starts_off);
  const void* const* ptrs = reinterpret_cast<const void* const*>(table + hdr->ptrs_off);
  const unsigned int n_tasks = hdr->n_tasks, total = hdr->total_chunks, chunk_elems = hdr->chunk_elems;

  __shared__ unsigned int s_idx[2];
  __shared__ unsigned int s_task;
  __shared__ double s_red[kThreads / 32];

  const unsigned int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  unsigned int cursor = 0;   // meaningful in warp 0
  int buf = 0;
  if (tid == 0) s_idx[0] = atomicAdd(&hdr->counter, 1u);
  __syncthreads();

  while (true) {
    const unsigned int idx = s_idx[buf];
    if (idx >= total) break;
    if (warp == 0) {
      // starts[] is increasing and starts[cursor] <= idx: advance 32 tasks at a time
      while (true) {
        const unsigned int probe = cursor + 1 + lane;
        const bool le = probe < n_tasks && __ldg(starts + probe) <= idx;
        const unsigned int adv = __popc(__ballot_sync(0xffffffffu, le));
        cursor += adv;
        if (adv < 32) break;
      }
      if (lane == 0) s_task = cursor;
    } else if (tid == kThreads - 1) {
      s_idx[buf ^ 1] = atomicAdd(&hdr->counter, 1u);
    }
    __syncthreads();

    const unsigned int t = s_task;
    const PsTaskDev* T = tasks + t;
    const unsigned int c = idx - T->first_chunk;
    const unsigned long long nelem = T->nelem;
    const size_t begin = (size_t)c * chunk_elems;
    const unsigned int count = (unsigned int)min((unsigned long long)chunk_elems, nelem - begin);
    const PsJobDev* J = jobs + T->job;
    Hp h;
    h.lr = J->lr; h.mom = J->mom; h.wd = J->wd; h.b1 = J->b1; h.b2 = J->b2;
    h.omb1 = J->omb1; h.omb2 = J->omb2; h.eps = J->eps; h.gs = J->gs;
    h.ss_t = T->ss_t; h.sbc2_t = T->sbc2_t;
    const int W = J->W;
    const void* const* shards = ptrs + T->shard_row;
    const bool vec_ok = T->vec_ok != 0;
    double sq = 0.0;
    const int kind = (J->opt << 1) | J->grad_dtype;
    switch (kind) {
      case 0: run_chunk<0, false>(h, shards, W, T->p, T->s0, T->s1, begin, count, vec_ok, sq); break;
      case 1: run_chunk<0, true>(h, shards, W, T->p, T->s0, T->s1, begin, count, vec_ok, sq); break;
      case 2: run_chunk<1, false>(h, shards, W, T->p, T->s0, T->s1, begin, count, vec_ok, sq); break;
      default: run_chunk<1, true>(h, shards, W, T->p, T->s0, T->s1, begin, count, vec_ok, sq); break;
    }

    // chunk sum of squares: lanes, then warps, in a fixed order
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sq += __shfl_down_sync(0xffffffffu, sq, o);
    if (lane == 0) s_red[warp] = sq;
    __syncthreads();
    if (tid == 0) {
      double s = s_red[0];
#pragma unroll
      for (int k = 1; k < kThreads / 32; ++k) s += s_red[k];
      const unsigned int first = T->first_chunk, n = T->nchunks;
      __stcg(partials + idx, s);
      __threadfence();
      const unsigned int done = atomicAdd(&tasks[t].ticket, 1u);
      if (done == n - 1) {
        __threadfence();
        double tot = 0.0;
        for (unsigned int k = 0; k < n; ++k) tot += __ldcg(partials + first + k);
        PsStat st;
        st.sqnorm = tot;
        st.step = T->step;
        stats[T->stat_idx] = st;
      }
    }
    buf ^= 1;
  }
}

}  // namespace psb
