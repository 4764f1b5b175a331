// CPU oracle for Parameter Service model aggregation.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
// CUDA library is checked against.  It shares no code, header, table or helper
// with the CUDA path and nothing in the product may call it.
//
// What it computes (paper, Section 2 "Background and Motivation": the server
// hosts the master copy and updates it using the aggregated result; Figure 1:
// all workers push, the server updates, workers pull; Appendix A: state is
// keyed by (job ID, tensor ID); Section 2.2 "Tensor-Based Model Structure":
// tensors are independent during aggregation).  The paper never prints the
// arithmetic of the update, so the canonical form below is this project's
// reading of it: the W pushed shards are SUMMED in worker order 0..W-1 and a
// textbook optimizer step is applied to the master copy.
//
// Canonical arithmetic, for one block at aggregate number t (t = 1 first):
//
//   G  = g_0[i];  for w = 1..W-1:  G = G + g_w[i]       (bf16 shard: bits<<16)
//   G  = G * grad_scale
//   d  = G + (wd * p[i])
//   SGD :  v' = (mom * v[i]) + d ;          p' = p[i] - (lr * v')
//   ADAM:  m' = (b1 * m[i]) + (omb1 * d)                omb1 = 1 - b1
//          v' = (b2 * v[i]) + (omb2 * (d * d))          omb2 = 1 - b2
//          den = (sqrt(v') / sbc2_t) + eps              sbc2_t = sqrt(1 - b2^t)
//          p' = p[i] - (ss_t * (m' / den))              ss_t   = lr / (1 - b1^t)
//   sqnorm = sum_i G*G   (always accumulated in binary64, sequentially)
//
// Two modes:
//   * binary32 mode ("f32"): every + - * / sqrt above is ONE IEEE-754 binary32
//     round-to-nearest-even operation, no fused multiply-add (build with
//     -ffp-contract=off), no flush-to-zero.  ss_t and sbc2_t are formed in
//     binary64 with pow() and rounded once to binary32.
//   * binary64 mode ("f64"): the same formulas with every quantity in binary64
//     (hyper-parameters are the binary32 values widened).  Used as the "truth"
//     the binary32 mode is compared with.
//
// The loops are the definition written out: blocks -> elements -> workers.
// There is no blocking, vectorisation or reordering.  OpenMP is used only
// ACROSS blocks in oracle_run_blocks (blocks are independent).
//
// Parity pins (tests/test_oracle_pins.py): W identical shards -> W*g; zero
// gradient + zero weight decay leaves p fixed; hand-worked 3-step momentum
// recurrence; geometric closed forms for momentum and weight decay; Adam first
// step and constant-gradient closed forms; bf16 widening over all 65,536 bit
// patterns; binary32 mode against binary64 mode.  The paper prints no worked
// aggregation example, so parity with the paper's own aggregator is unpinned;
// parity is with the definition above.

#include <cmath>
#include <cstddef>
#include <cstdint>
#include <cstring>

#ifdef _OPENMP
#include <omp.h>
#endif

extern "C" {

enum { ORACLE_SGD = 0, ORACLE_ADAM = 1 };
enum { ORACLE_F32 = 0, ORACLE_BF16 = 1 };

typedef struct {
  int32_t opt;          // ORACLE_SGD | ORACLE_ADAM
  int32_t grad_dtype;   // ORACLE_F32 | ORACLE_BF16
  int32_t num_workers;  // W >= 1
  float lr, momentum, weight_decay, beta1, beta2, eps, grad_scale;
} oracle_hparams;

// One block's aggregation task.  `shards` points at W pointers, each to nelem
// contiguous gradient values (float or bf16 bit patterns).  p/s0/s1 are
// updated in place: s0 = momentum (SGD) or first moment (Adam); s1 = second
// moment (Adam only, may be null for SGD).  In f64 mode p/s0/s1 are double*.
typedef struct {
  oracle_hparams hp;
  uint64_t step;        // t, the number of this aggregate (>= 1)
  uint64_t nelem;
  const void* const* shards;
  void* p;
  void* s0;
  void* s1;
  double sqnorm;        // out
} oracle_task;

// Exact widening of a bf16 bit pattern to binary32: the 16 bits become the
// upper half of the binary32 word.
float oracle_bf16_to_f32(uint16_t bits) {
  uint32_t u = (uint32_t)bits << 16;
  float f;
  std::memcpy(&f, &u, sizeof f);
  return f;
}

// Array form of the widening (results stored to memory, so NaN payloads keep
// their bits).
void oracle_widen_bf16(const uint16_t* bits, float* out, uint64_t n) {
  for (uint64_t i = 0; i < n; ++i) out[i] = oracle_bf16_to_f32(bits[i]);
}

static inline float shard_value(const oracle_hparams* hp, const void* shard, uint64_t i) {
  if (hp->grad_dtype == ORACLE_BF16)
    return oracle_bf16_to_f32(((const uint16_t*)shard)[i]);
  return ((const float*)shard)[i];
}

// Bias-correction scalars of Adam at step t, formed in binary64.
double oracle_adam_step_size(float lr, float beta1, uint64_t t) {
  return (double)lr / (1.0 - std::pow((double)beta1, (double)t));
}
double oracle_adam_sqrt_bc2(float beta2, uint64_t t) {
  return std::sqrt(1.0 - std::pow((double)beta2, (double)t));
}

static int check_task(const oracle_task* k) {
  if (!k || !k->shards || !k->p || !k->s0) return -1;
  if (k->hp.num_workers < 1 || k->step < 1) return -1;
  if (k->hp.opt != ORACLE_SGD && k->hp.opt != ORACLE_ADAM) return -1;
  if (k->hp.grad_dtype != ORACLE_F32 && k->hp.grad_dtype != ORACLE_BF16) return -1;
  if (k->hp.opt == ORACLE_ADAM && !k->s1) return -1;
  for (int w = 0; w < k->hp.num_workers; ++w)
    if (!k->shards[w]) return -1;
  return 0;
}

// binary32 mode.
int oracle_block_step_f32(oracle_task* k) {
  if (check_task(k)) return -1;
  const oracle_hparams* hp = &k->hp;
  const int W = hp->num_workers;
  float* p = (float*)k->p;
  float* s0 = (float*)k->s0;
  float* s1 = (float*)k->s1;
  const float lr = hp->lr, mom = hp->momentum, wd = hp->weight_decay;
  const float b1 = hp->beta1, b2 = hp->beta2, eps = hp->eps, gs = hp->grad_scale;
  const float omb1 = 1.0f - b1;
  const float omb2 = 1.0f - b2;
  const float ss_t = (float)oracle_adam_step_size(lr, b1, k->step);
  const float sbc2_t = (float)oracle_adam_sqrt_bc2(b2, k->step);
  double sq = 0.0;
  for (uint64_t i = 0; i < k->nelem; ++i) {
    float G = shard_value(hp, k->shards[0], i);
    for (int w = 1; w < W; ++w) G = G + shard_value(hp, k->shards[w], i);
    G = G * gs;
    sq += (double)G * (double)G;
    const float wdp = wd * p[i];
    const float d = G + wdp;
    if (hp->opt == ORACLE_SGD) {
      const float mv = mom * s0[i];
      const float v = mv + d;
      const float step = lr * v;
      s0[i] = v;
      p[i] = p[i] - step;
    } else {
      const float b1m = b1 * s0[i];
      const float od = omb1 * d;
      const float m = b1m + od;
      const float dd = d * d;
      const float b2v = b2 * s1[i];
      const float odd = omb2 * dd;
      const float v = b2v + odd;
      const float r = std::sqrt(v);   // sqrtss: correctly rounded binary32
      const float rh = r / sbc2_t;
      const float den = rh + eps;
      const float q = m / den;
      const float step = ss_t * q;
      s0[i] = m;
      s1[i] = v;
      p[i] = p[i] - step;
    }
  }
  k->sqnorm = sq;
  return 0;
}

// binary64 mode: same formulas, every quantity in binary64.
int oracle_block_step_f64(oracle_task* k) {
  if (check_task(k)) return -1;
  const oracle_hparams* hp = &k->hp;
  const int W = hp->num_workers;
  double* p = (double*)k->p;
  double* s0 = (double*)k->s0;
  double* s1 = (double*)k->s1;
  const double lr = hp->lr, mom = hp->momentum, wd = hp->weight_decay;
  const double b1 = hp->beta1, b2 = hp->beta2, eps = hp->eps, gs = hp->grad_scale;
  const double omb1 = 1.0 - b1;
  const double omb2 = 1.0 - b2;
  const double ss_t = oracle_adam_step_size(hp->lr, hp->beta1, k->step);
  const double sbc2_t = oracle_adam_sqrt_bc2(hp->beta2, k->step);
  double sq = 0.0;
  for (uint64_t i = 0; i < k->nelem; ++i) {
    double G = (double)shard_value(hp, k->shards[0], i);
    for (int w = 1; w < W; ++w) G = G + (double)shard_value(hp, k->shards[w], i);
    G = G * gs;
    sq += G * G;
    const double d = G + wd * p[i];
    if (hp->opt == ORACLE_SGD) {
      const double v = mom * s0[i] + d;
      s0[i] = v;
      p[i] = p[i] - lr * v;
    } else {
      const double m = b1 * s0[i] + omb1 * d;
      const double v = b2 * s1[i] + omb2 * (d * d);
      const double den = std::sqrt(v) / sbc2_t + eps;
      s0[i] = m;
      s1[i] = v;
      p[i] = p[i] - ss_t * (m / den);
    }
  }
  k->sqnorm = sq;
  return 0;
}

// Runs n independent block tasks (binary32 mode), OpenMP across blocks only.
// Returns the number of threads used, or -1 if any task was malformed.
int oracle_run_blocks(oracle_task* tasks, int n, int nthreads) {
  int bad = 0;
  int used = 1;
#ifdef _OPENMP
  if (nthreads < 1) nthreads = omp_get_max_threads();
  used = nthreads;
#pragma omp parallel for schedule(dynamic, 1) num_threads(nthreads) reduction(| : bad)
#endif
  for (int b = 0; b < n; ++b) bad |= (oracle_block_step_f32(&tasks[b]) != 0);
  (void)nthreads;
  return bad ? -1 : used;
}

int oracle_hardware_threads(void) {
#ifdef _OPENMP
  return omp_get_num_procs();
#else
  return 1;
#endif
}

}  // extern "C"
