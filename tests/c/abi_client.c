/* A plain C99 client of the library: proves that the boundary needs neither C++
 * nor Python.  Uses a planning-only service (no device), so it runs anywhere:
 * registers two jobs, pushes pointers, asks for the packed table of a ready
 * list and checks the bookkeeping rules.  Exit code 0 = all checks passed. */
#include <stdio.h>
#include <string.h>

#include "ps_b200.h"

#define CHECK(cond)                                                        \
  do {                                                                     \
    if (!(cond)) {                                                         \
      fprintf(stderr, "check failed at line %d: %s\n", __LINE__, #cond);   \
      return 1;                                                            \
    }                                                                      \
  } while (0)

int main(void) {
  ps_service* svc = NULL;
  ps_job_desc sgd, adam;
  ps_task ready[3];
  ps_chunk_info chunks[64];
  size_t n_chunks = 0, used = 0, largest = 0, packed = 0;
  unsigned long long step = 99;
  static float shard[4096];
  const float* params = NULL;
  int job0 = -1, job1 = -1, w;
  long long opt = -1;

  CHECK(strstr(ps_version(), "sm_100a") != NULL);
  CHECK(ps_create(&svc, PS_DEVICE_NONE, 2, (size_t)1 << 24) == PS_OK);

  memset(&sgd, 0, sizeof sgd);
  sgd.opt = PS_SGD; sgd.grad_dtype = PS_F32; sgd.num_workers = 3;
  sgd.lr = 0.1f; sgd.momentum = 0.9f; sgd.weight_decay = 1e-4f; sgd.grad_scale = 1.0f;
  adam = sgd;
  adam.opt = PS_ADAM; adam.grad_dtype = PS_BF16; adam.num_workers = 2;
  adam.beta1 = 0.9f; adam.beta2 = 0.999f; adam.eps = 1e-8f;
  CHECK(ps_register_job(svc, &sgd, &job0) == PS_OK && job0 == 0);
  CHECK(ps_register_job(svc, &adam, &job1) == PS_OK && job1 == 1);
  sgd.num_workers = 0;
  CHECK(ps_register_job(svc, &sgd, &job0) == PS_ERR_BAD_ARG);
  job0 = 0;

  CHECK(ps_register_block(svc, job0, 0, 20000, 0, NULL) == PS_OK);
  CHECK(ps_register_block(svc, job0, 1, 7, 1, NULL) == PS_OK);
  CHECK(ps_register_block(svc, job1, 0, 4096, 1, NULL) == PS_OK);
  CHECK(ps_register_block(svc, job0, 0, 20000, 0, NULL) == PS_ERR_DUPLICATE);
  CHECK(ps_arena_info(svc, 0, &used, &largest) == PS_OK && used == 2 * 80128);   /* p | momentum, 256-byte sections */
  CHECK(ps_block_export(svc, job1, 0, NULL, 0, &packed, &step, NULL) == PS_OK);
  CHECK(packed == 3 * 16384 && step == 0);                                       /* p | m | v */

  for (w = 0; w < 3; ++w) CHECK(ps_push(svc, job0, 0, w, shard) == PS_OK);
  CHECK(ps_push(svc, job0, 0, 1, shard) == PS_ERR_DUPLICATE);
  CHECK(ps_push(svc, job0, 0, 3, shard) == PS_ERR_BAD_ARG);
  CHECK(ps_push(svc, job1, 0, 0, (const char*)shard + 1) == PS_ERR_ALIGN);
  CHECK(ps_push(svc, job1, 0, 0, shard) == PS_OK);

  ready[0].job = job0; ready[0].block = 0;
  ready[1].job = job1; ready[1].block = 0;
  CHECK(ps_plan(svc, ready, 2, chunks, 64, &n_chunks) == PS_ERR_NOT_READY);       /* job1 lacks a push */
  CHECK(ps_push(svc, job1, 0, 1, shard) == PS_OK);
  CHECK(ps_plan(svc, ready, 2, chunks, 64, &n_chunks) == PS_OK && n_chunks >= 2);
  {
    unsigned long long elems0 = 0, elems1 = 0;
    size_t i;
    for (i = 0; i < n_chunks; ++i) {
      if (chunks[i].job == job0) elems0 += chunks[i].elem_count; else elems1 += chunks[i].elem_count;
      CHECK(chunks[i].num_workers == (chunks[i].job == job0 ? 3 : 2));
    }
    CHECK(elems0 == 20000 && elems1 == 4096);
  }
  ready[2] = ready[0];
  CHECK(ps_plan(svc, ready, 3, chunks, 64, &n_chunks) == PS_ERR_DUPLICATE);

  /* no device: nothing computes, nothing pretends to */
  CHECK(ps_aggregate(svc, ready, 2, NULL) == PS_ERR_NO_DEVICE);
  CHECK(ps_pull(svc, job0, 0, &params) == PS_ERR_NO_DEVICE);
  CHECK(ps_migrate_block(svc, job0, 0, 1, NULL) == PS_ERR_NO_DEVICE);

  CHECK(ps_set_option(svc, PS_OPT_CHUNK_ELEMS, 1000) == PS_ERR_BAD_ARG);
  CHECK(ps_set_option(svc, PS_OPT_CHUNK_ELEMS, 2048) == PS_OK);
  CHECK(ps_get_option(svc, PS_OPT_CHUNK_ELEMS, &opt) == PS_OK && opt == 2048);
  CHECK(ps_get_option(svc, PS_OPT_INLINE_TABLE, &opt) == PS_OK && opt == 1);

  CHECK(ps_unregister_block(svc, job0, 1) == PS_OK);
  CHECK(ps_arena_info(svc, 1, &used, &largest) == PS_OK && used == 3 * 16384);
  CHECK(ps_unregister_block(svc, job0, 1) == PS_ERR_BAD_ARG);
  CHECK(strlen(ps_strerror(PS_ERR_NOT_READY)) > 0);
  CHECK(ps_destroy(svc) == PS_OK);
  CHECK(ps_destroy(NULL) == PS_ERR_BAD_HANDLE);
  puts("abi_client: ok");
  return 0;
}
