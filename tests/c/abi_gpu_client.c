/* A plain C99 client that computes on the GPU through the library alone (CUDA
 * runtime for memory, no Python, no C++): one SGD job, W = 4 identical shards
 * of value 0.25, two iterations, checked against the hand-worked momentum
 * recurrence  G = 1,  v = 1, 1.5,  p = p0 - 0.5, p0 - 1.25  (lr 0.5, momentum
 * 0.5, no decay) and the block statistic sum G*G = nelem.
 * Exit code 0 = all checks passed. */
#include <stdio.h>
#include <stdlib.h>

#include <cuda_runtime_api.h>

#include "ps_b200.h"

#define CHECK(cond)                                                        \
  do {                                                                     \
    if (!(cond)) {                                                         \
      fprintf(stderr, "check failed at line %d: %s\n", __LINE__, #cond);   \
      return 1;                                                            \
    }                                                                      \
  } while (0)

int main(void) {
  const size_t n = 100003;                 /* several chunks and a ragged tail */
  const int W = 4;
  ps_service* svc = NULL;
  ps_job_desc d;
  ps_task task;
  float *host, *grads[4];
  const float* params = NULL;
  double sq = 0.0;
  unsigned long long step = 0;
  int job = -1, w, it;
  size_t i;

  CHECK(cudaSetDevice(0) == cudaSuccess);
  CHECK(ps_create(&svc, 0, 1, (size_t)8 << 20) == PS_OK);
  d.opt = PS_SGD; d.grad_dtype = PS_F32; d.num_workers = W;
  d.lr = 0.5f; d.momentum = 0.5f; d.weight_decay = 0.0f;
  d.beta1 = 0.0f; d.beta2 = 0.0f; d.eps = 0.0f; d.grad_scale = 1.0f;
  CHECK(ps_register_job(svc, &d, &job) == PS_OK);

  host = (float*)malloc(n * sizeof(float));
  CHECK(host != NULL);
  for (i = 0; i < n; ++i) host[i] = 0.5f * (float)(i % 1024);
  CHECK(ps_register_block(svc, job, 0, n, 0, host) == PS_OK);      /* initial parameters from host memory */

  for (i = 0; i < n; ++i) host[i] = 0.25f;
  for (w = 0; w < W; ++w) {
    CHECK(cudaMalloc((void**)&grads[w], n * sizeof(float)) == cudaSuccess);
    CHECK(cudaMemcpy(grads[w], host, n * sizeof(float), cudaMemcpyHostToDevice) == cudaSuccess);
  }
  task.job = job; task.block = 0;
  for (it = 0; it < 2; ++it) {
    for (w = 0; w < W; ++w) CHECK(ps_push(svc, job, 0, w, grads[w]) == PS_OK);
    CHECK(ps_aggregate(svc, &task, 1, NULL) == PS_OK);
    CHECK(ps_pull(svc, job, 0, &params) == PS_OK);
    CHECK(cudaDeviceSynchronize() == cudaSuccess);
    CHECK(cudaMemcpy(host, params, n * sizeof(float), cudaMemcpyDeviceToHost) == cudaSuccess);
    for (i = 0; i < n; ++i) {
      const float want = 0.5f * (float)(i % 1024) - (it == 0 ? 0.5f : 1.25f);   /* exact in binary32 */
      if (host[i] != want) {
        fprintf(stderr, "iteration %d element %lu: got %.9g want %.9g\n", it, (unsigned long)i, host[i], want);
        return 1;
      }
    }
    CHECK(ps_block_stats(svc, job, 0, &sq, &step) == PS_OK);
    CHECK(sq == (double)n && step == (unsigned long long)(it + 1));
  }
  for (w = 0; w < W; ++w) CHECK(cudaFree(grads[w]) == cudaSuccess);
  free(host);
  CHECK(ps_destroy(svc) == PS_OK);
  puts("abi_gpu_client: ok");
  return 0;
}
