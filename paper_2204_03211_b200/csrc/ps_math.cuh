// Arithmetic of one aggregation (defined operation by operation in
// include/ps_b200.h) and the chunk bodies that read gradients straight from
// global memory.  Explicit round-to-nearest intrinsics keep the compiler from
// fusing multiply-adds, so the binary32 result is unique.
#pragma once

#include "ps_types.cuh"

namespace psb {

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

// lo += bf16(low half of u), hi += bf16(high half of u).  The mixed-precision
// add widens its bf16 operand exactly and rounds the binary32 sum once to
// nearest-even (subnormals kept), i.e. the same bits as
// __fadd_rn(acc, bf16_lo/hi(u)) with one instruction per element instead of two.
__device__ __forceinline__ void add_bf16x2(float& lo, float& hi, unsigned int u) {
  asm("{\n\t"
      ".reg .b16 l, h;\n\t"
      "mov.b32 {l, h}, %2;\n\t"
      "add.rn.f32.bf16 %0, l, %0;\n\t"
      "add.rn.f32.bf16 %1, h, %1;\n\t"
      "}"
      : "+f"(lo), "+f"(hi)
      : "r"(u));
}

// Shard pointer w of a task (uniform across the CTA).  A generic load: the
// pointer row may sit in the global task table or in shared memory.
__device__ __forceinline__ const void* ld_ptr(const void* const* shards, int w = 0) {
  return shards[w];
}

// Streaming (read-once) 128-bit load.
__device__ __forceinline__ uint4 ld_stream(const void* p) { return __ldcs(reinterpret_cast<const uint4*>(p)); }

__device__ __forceinline__ float4 as_f4(const uint4& t) {
  return make_float4(__uint_as_float(t.x), __uint_as_float(t.y), __uint_as_float(t.z), __uint_as_float(t.w));
}

__device__ __forceinline__ float4 add4(float4 a, uint4 b) {
  a.x = __fadd_rn(a.x, __uint_as_float(b.x));
  a.y = __fadd_rn(a.y, __uint_as_float(b.y));
  a.z = __fadd_rn(a.z, __uint_as_float(b.z));
  a.w = __fadd_rn(a.w, __uint_as_float(b.w));
  return a;
}

__device__ __forceinline__ void widen8(const uint4& t, float (&o)[8]) {
  o[0] = bf16_lo(t.x); o[1] = bf16_hi(t.x); o[2] = bf16_lo(t.y); o[3] = bf16_hi(t.y);
  o[4] = bf16_lo(t.z); o[5] = bf16_hi(t.z); o[6] = bf16_lo(t.w); o[7] = bf16_hi(t.w);
}

// Updates four consecutive elements starting at e and stores them.
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
// NT = number of cooperating threads, tid = this thread's index among them.
//
// The vector bodies are bound by memory latency, not by issue slots: a thread
// cannot hold enough 128-bit loads in registers to cover the HBM latency at
// full occupancy.  So lines are requested ahead of their use with L2
// prefetches, which occupy no register: the demand loads then complete from
// L2.  One lane per 128-byte line issues the prefetch; every prefetched
// address is one that a demand load of the same chunk reads later.

__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

constexpr int kAheadF32 = 2;         // fp32 shards: workers requested ahead inside the worker loop
constexpr int kAheadBf16 = 4;        // bf16 shards: the same
constexpr int kNextTripMaxW = 8;     // up to this many workers the loop is too short to run ahead in: the
                                     // next trip's first lines are requested at the top of each trip instead

// fp32 gradients, 16-byte aligned: each thread owns U float4 groups per trip.
template <int OPT, int U, int NT>
__device__ __forceinline__ void chunk_f32_vec(unsigned int tid, const Hp& h, const void* const* __restrict__ shards,
                                              int W, float* __restrict__ p, float* __restrict__ s0,
                                              float* __restrict__ s1, size_t begin, unsigned int count, double& sq) {
  const unsigned int nvec = count >> 2;
  const bool pf_lane = (tid & 7) == 0;      // 8 lanes x 16 bytes = one line
  unsigned int i = tid;
  // full trips: U groups per thread, no predicates
  for (; i + (U - 1) * NT < nvec; i += U * NT) {
    float4 acc[U], pv[U], av[U], bv[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const size_t e = begin + 4 * (size_t)(i + u * NT);
      pv[u] = *reinterpret_cast<const float4*>(p + e);
      av[u] = *reinterpret_cast<const float4*>(s0 + e);
      if (OPT == 1) bv[u] = *reinterpret_cast<const float4*>(s1 + e); else bv[u] = make_float4(0, 0, 0, 0);
    }
    if (pf_lane) {
      if (W <= kNextTripMaxW && i + U * NT + (U - 1) * NT < nvec) {
        // next full trip: parameters, state and the first shards
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const size_t e = begin + 4 * (size_t)(i + (U + u) * NT);
          prefetch_l2(p + e);
          prefetch_l2(s0 + e);
          if (OPT == 1) prefetch_l2(s1 + e);
        }
        for (int w = 0; w <= kAheadF32 && w < W; ++w) {
          const float* g = static_cast<const float*>(ld_ptr(shards, w));
#pragma unroll
          for (int u = 0; u < U; ++u) prefetch_l2(g + begin + 4 * (size_t)(i + (U + u) * NT));
        }
      }
      if (W > kNextTripMaxW || i == tid) {
        // this trip's first shards after shard 0 (not requested by an earlier trip)
        for (int w = 1; w <= kAheadF32 && w < W; ++w) {
          const float* g = static_cast<const float*>(ld_ptr(shards, w));
#pragma unroll
          for (int u = 0; u < U; ++u) prefetch_l2(g + begin + 4 * (size_t)(i + u * NT));
        }
      }
    }
    {
      const float* g = static_cast<const float*>(ld_ptr(shards));
#pragma unroll
      for (int u = 0; u < U; ++u) acc[u] = as_f4(ld_stream(g + begin + 4 * (size_t)(i + u * NT)));
    }
#pragma unroll 2
    for (int w = 1; w < W; ++w) {
      if (pf_lane && w + kAheadF32 < W) {
        const float* ga = static_cast<const float*>(ld_ptr(shards, w + kAheadF32));
#pragma unroll
        for (int u = 0; u < U; ++u) prefetch_l2(ga + begin + 4 * (size_t)(i + u * NT));
      }
      const float* g = static_cast<const float*>(ld_ptr(shards, w));
#pragma unroll
      for (int u = 0; u < U; ++u) acc[u] = add4(acc[u], ld_stream(g + begin + 4 * (size_t)(i + u * NT)));
    }
#pragma unroll
    for (int u = 0; u < U; ++u)
      update4<OPT>(h, acc[u], p, s0, s1, begin + 4 * (size_t)(i + u * NT), pv[u], av[u], bv[u], sq);
  }
  // remaining groups, one per thread
  for (; i < nvec; i += NT) {
    const size_t e = begin + 4 * (size_t)i;
    const float4 pv = *reinterpret_cast<const float4*>(p + e);
    const float4 av = *reinterpret_cast<const float4*>(s0 + e);
    const float4 bv = (OPT == 1) ? *reinterpret_cast<const float4*>(s1 + e) : make_float4(0, 0, 0, 0);
    float4 acc = as_f4(ld_stream(static_cast<const float*>(ld_ptr(shards)) + e));
#pragma unroll 4
    for (int w = 1; w < W; ++w) acc = add4(acc, ld_stream(static_cast<const float*>(ld_ptr(shards, w)) + e));
    update4<OPT>(h, acc, p, s0, s1, e, pv, av, bv, sq);
  }
}

// bf16 gradients, 16-byte aligned: each thread owns 8 consecutive elements.
// Parameters and state are requested at the top of a trip and loaded after the
// worker loop, so their 24 registers are free while the shards stream.
template <int OPT, int NT>
__device__ __forceinline__ void chunk_bf16_vec(unsigned int tid, const Hp& h, const void* const* __restrict__ shards,
                                               int W, float* __restrict__ p, float* __restrict__ s0,
                                               float* __restrict__ s1, size_t begin, unsigned int count, double& sq) {
  const unsigned int nvec = count >> 3;
  const bool pf_lane = (tid & 7) == 0;      // shards: 8 lanes x 16 bytes = one line
  for (unsigned int i = tid; i < nvec; i += NT) {
    const size_t e = begin + 8 * (size_t)i;
    if ((tid & 3) == 0) {                   // parameters and state: 4 lanes x 32 bytes = one line
      prefetch_l2(p + e);
      prefetch_l2(s0 + e);
      if (OPT == 1) prefetch_l2(s1 + e);
    }
    if (pf_lane)
      for (int w = 1; w <= kAheadBf16 && w < W; ++w)
        prefetch_l2(static_cast<const unsigned short*>(ld_ptr(shards, w)) + e);
    float acc[8];
    widen8(ld_stream(static_cast<const unsigned short*>(ld_ptr(shards)) + e), acc);
#pragma unroll 4
    for (int w = 1; w < W; ++w) {
      if (pf_lane && w + kAheadBf16 < W)
        prefetch_l2(static_cast<const unsigned short*>(ld_ptr(shards, w + kAheadBf16)) + e);
      const uint4 t = ld_stream(static_cast<const unsigned short*>(ld_ptr(shards, w)) + e);
      add_bf16x2(acc[0], acc[1], t.x);
      add_bf16x2(acc[2], acc[3], t.y);
      add_bf16x2(acc[4], acc[5], t.z);
      add_bf16x2(acc[6], acc[7], t.w);
    }
    const float4 p0 = *reinterpret_cast<const float4*>(p + e), p1 = *reinterpret_cast<const float4*>(p + e + 4);
    const float4 a0 = *reinterpret_cast<const float4*>(s0 + e), a1 = *reinterpret_cast<const float4*>(s0 + e + 4);
    float4 b0 = make_float4(0, 0, 0, 0), b1 = b0;
    if (OPT == 1) {
      b0 = *reinterpret_cast<const float4*>(s1 + e);
      b1 = *reinterpret_cast<const float4*>(s1 + e + 4);
    }
    update4<OPT>(h, make_float4(acc[0], acc[1], acc[2], acc[3]), p, s0, s1, e, p0, a0, b0, sq);
    update4<OPT>(h, make_float4(acc[4], acc[5], acc[6], acc[7]), p, s0, s1, e + 4, p1, a1, b1, sq);
  }
}

// Any alignment, any count: one element per thread per trip, elements [first, count).
template <int OPT, bool BF16, int NT>
__device__ __forceinline__ void chunk_scalar(unsigned int tid, const Hp& h, const void* const* __restrict__ shards,
                                             int W, float* __restrict__ p, float* __restrict__ s0,
                                             float* __restrict__ s1, size_t begin, unsigned int first,
                                             unsigned int count, double& sq) {
  for (unsigned int i = first + tid; i < count; i += NT) {
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

template <int OPT, bool BF16, int NT>
__device__ __forceinline__ void run_chunk(unsigned int tid, const Hp& h, const void* const* shards, int W, float* p,
                                          float* s0, float* s1, size_t begin, unsigned int count, bool vec_ok,
                                          double& sq) {
  if (vec_ok) {
    constexpr unsigned int V = BF16 ? 8 : 4;
    const unsigned int body = count & ~(V - 1);
    if (BF16) chunk_bf16_vec<OPT, NT>(tid, h, shards, W, p, s0, s1, begin, body, sq);
    else chunk_f32_vec<OPT, 2, NT>(tid, h, shards, W, p, s0, s1, begin, body, sq);
    if (body != count) chunk_scalar<OPT, BF16, NT>(tid, h, shards, W, p, s0, s1, begin, body, count, sq);
  } else {
    chunk_scalar<OPT, BF16, NT>(tid, h, shards, W, p, s0, s1, begin, 0, count, sq);
  }
}

__device__ __forceinline__ Hp load_hp(const PsJobDev* J, const PsTaskDev* T) {
  Hp h;
  h.lr = J->lr; h.mom = J->mom; h.wd = J->wd; h.b1 = J->b1; h.b2 = J->b2;
  h.omb1 = J->omb1; h.omb2 = J->omb2; h.eps = J->eps; h.gs = J->gs;
  h.ss_t = T->ss_t; h.sbc2_t = T->sbc2_t;
  return h;
}

// One chunk read with ordinary loads; dispatches on (optimizer, gradient type).
struct JobView {                       // what a chunk body needs from its job, loaded once
  Hp h;
  int W, kind;                         // kind = (optimizer << 1) | gradient type
};

__device__ __forceinline__ JobView load_job(const PsJobDev* J, const PsTaskDev* T) {
  JobView v;
  v.h = load_hp(J, T);
  v.W = J->W;
  v.kind = (J->opt << 1) | J->grad_dtype;
  return v;
}

template <int NT>
__device__ __forceinline__ void run_chunk_view(unsigned int tid, const JobView& v, const PsTaskDev* T,
                                               const void* const* shards, size_t begin, unsigned int count,
                                               double& sq) {
  const Hp& h = v.h;
  const int W = v.W;
  const bool vec_ok = T->vec_ok != 0;
  switch (v.kind) {
    case 0: run_chunk<0, false, NT>(tid, h, shards, W, T->p, T->s0, T->s1, begin, count, vec_ok, sq); break;
    case 1: run_chunk<0, true, NT>(tid, h, shards, W, T->p, T->s0, T->s1, begin, count, vec_ok, sq); break;
    case 2: run_chunk<1, false, NT>(tid, h, shards, W, T->p, T->s0, T->s1, begin, count, vec_ok, sq); break;
    default: run_chunk<1, true, NT>(tid, h, shards, W, T->p, T->s0, T->s1, begin, count, vec_ok, sq); break;
  }
}

template <int NT>
__device__ __forceinline__ void run_chunk_any(unsigned int tid, const PsJobDev* J, const PsTaskDev* T,
                                              const void* const* shards, size_t begin, unsigned int count,
                                              double& sq) {
  const Hp h = load_hp(J, T);
  const int W = J->W;
  const bool vec_ok = T->vec_ok != 0;
  switch ((J->opt << 1) | J->grad_dtype) {
    case 0: run_chunk<0, false, NT>(tid, h, shards, W, T->p, T->s0, T->s1, begin, count, vec_ok, sq); break;
    case 1: run_chunk<0, true, NT>(tid, h, shards, W, T->p, T->s0, T->s1, begin, count, vec_ok, sq); break;
    case 2: run_chunk<1, false, NT>(tid, h, shards, W, T->p, T->s0, T->s1, begin, count, vec_ok, sq); break;
    default: run_chunk<1, true, NT>(tid, h, shards, W, T->p, T->s0, T->s1, begin, count, vec_ok, sq); break;
  }
}

// Sum of n partial sums of squares in a FIXED order, by one warp: lane l adds
// the partials l, l+32, l+64, ... in increasing order, then the lanes are
// combined by a shuffle tree.  The result does not depend on which CTA produced
// which partial nor on arrival order.  (A single thread walking the list costs
// one L2 round trip per few partials: about 10 us for the 576 chunks of a
// 590 K-element tensor, which was most of such a launch's duration.)
__device__ __forceinline__ double sum_partials_warp(const double* partials, unsigned int n, unsigned int lane) {
  double tot = 0.0;
  for (unsigned int k = lane; k < n; k += 32) tot += __ldcg(partials + k);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) tot += __shfl_down_sync(0xffffffffu, tot, o);
  return tot;     // complete in lane 0
}

// Publishes one partial sum of squares of a chunk (slot = chunk * parts + part)
// and, in the warp that delivers the task's last partial, adds all of the
// task's partials in the fixed order above.  Called by all 32 lanes of one warp
// per partial; `s` is taken from lane 0.
__device__ __forceinline__ void publish_part(PsTaskDev* tasks, unsigned int t, unsigned int slot, unsigned int parts,
                                             double s, PsStat* stats, double* partials, unsigned int lane) {
  const PsTaskDev* T = tasks + t;
  const unsigned int first = T->first_chunk * parts, n = T->nchunks * parts;
  unsigned int done = 0;
  if (lane == 0) {
    __stcg(partials + slot, s);
    __threadfence();
    done = atomicAdd(&tasks[t].ticket, 1u);
    __threadfence();
  }
  done = __shfl_sync(0xffffffffu, done, 0);
  if (done != n - 1) return;
  const double tot = sum_partials_warp(partials + first, n, lane);
  if (lane == 0) {
    PsStat st;
    st.sqnorm = tot;
    st.step = T->step;
    st.busy_ns = __ldcg(&T->busy_ns);
    const unsigned long long tf = __ldcg(&T->t_first);
    st.t_first = (tf == ~0ull) ? 0ull : tf;
    st.t_last = __ldcg(&T->t_last);
    st._r0 = 0;
    stats[T->stat_idx] = st;
  }
}

// The same for ONE calling thread, which adds the partials in chunk order itself.
// For the persistent kernel: a task there has at most a few
// hundred chunks, the other CTAs keep streaming while one thread adds, and keeping
// the other 31 lanes of the warp out of it keeps the chunk loop's registers free.
__device__ __forceinline__ void publish_one(PsTaskDev* tasks, unsigned int t, unsigned int slot, double s,
                                            PsStat* stats, double* partials) {
  const PsTaskDev* T = tasks + t;
  const unsigned int n = T->nchunks;
  const double* mine = partials + T->first_chunk;
  __stcg(partials + slot, s);
  __threadfence();
  if (atomicAdd(&tasks[t].ticket, 1u) != n - 1) return;
  __threadfence();
  double tot = 0.0;
  for (unsigned int k = 0; k < n; ++k) tot += __ldcg(mine + k);     // (unrolled, it spilled in the chunk loop: -3 %)
  PsStat st;
  st.sqnorm = tot;
  st.step = T->step;
  st.busy_ns = __ldcg(&T->busy_ns);
  const unsigned long long tf = __ldcg(&T->t_first);
  st.t_first = (tf == ~0ull) ? 0ull : tf;
  st.t_last = __ldcg(&T->t_last);
  st._r0 = 0;
  stats[T->stat_idx] = st;
}

__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// Adds one chunk's device time to its task's profile (before publish_part, whose
// fence orders these updates ahead of the ticket).
__device__ __forceinline__ void profile_chunk(PsTaskDev* T, unsigned long long t0, unsigned long long t1) {
  atomicAdd(&T->busy_ns, t1 - t0);
  atomicMin(&T->t_first, t0);
  atomicMax(&T->t_last, t1);
}

// Completion signal of a launch.  Every thread of a CTA calls this when the CTA
// has no more work.  The CTA that leaves last (counted in *exited, which it
// clears for the next launch that uses the same counter) stores `seq` to
// *done_word — a word in page-locked host memory that the host polls instead of
// recording and querying an event per launch.
// Ordering: the barrier puts the CTA's stores before thread 0's fence, which is
// cumulative, so they are visible device-wide before the CTA is counted; the
// last CTA's own fence does the same for the counts it has seen before it
// issues the store.  Whoever acts on the word is a later launch on this device
// (or a copy engine reading device memory), for which device-wide visibility is
// what counts; a system-wide fence here cost 1.4 us of every small launch
// (measured) and bought nothing for such readers.
// done_word == nullptr: the launch does not signal.
__device__ __forceinline__ void signal_exit(unsigned int* exited, unsigned long long* done_word,
                                            unsigned long long seq) {
  if (!done_word) return;
  __syncthreads();
  if (threadIdx.x != 0) return;
  __threadfence();
  if (atomicAdd(exited, 1u) != gridDim.x - 1) return;
  *exited = 0;
  __threadfence();
  *reinterpret_cast<volatile unsigned long long*>(done_word) = seq;
}

// Programmatic dependent launch: lets the next launch of the stream start its
// prologue while this one runs (a no-op for launches without the attribute) ...
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;"); }
// ... and waits until the launches this one depends on have completed and their
// stores are visible (returns at once when there is no such dependency).
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Advances `cursor` (uniform in the calling warp) to the task that owns chunk
// idx: starts[] is increasing and starts[cursor] <= idx on entry.
__device__ __forceinline__ unsigned int find_task(const unsigned int* starts, unsigned int n_tasks,
                                                  unsigned int cursor, unsigned int idx, unsigned int lane) {
  while (true) {
    const unsigned int probe = cursor + 1 + lane;
    const bool le = probe < n_tasks && __ldg(starts + probe) <= idx;
    const unsigned int adv = __popc(__ballot_sync(0xffffffffu, le));
    cursor += adv;
    if (adv < 32) break;
  }
  return cursor;
}

}  // namespace psb
