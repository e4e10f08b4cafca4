/*
 * Plain C use of the library: one small Expand-and-Prune rollout (2 groups of 16 trajectories
 * pruned to 8 at step 3 of 10, 4x32x32 latents) with no Python and no torch.  Device memory comes
 * from cudaMalloc; initial latents and the stand-in predictions are drawn with the library's own
 * generator (noise streams 1 and 2).  Prints the advantages and returns 0 if every group's
 * advantages sum to zero.
 *
 *   gcc abi_example.c -I../../include -I/usr/local/cuda/include -L.. -lprogrpo \
 *       -L/usr/local/cuda/lib64 -lcudart -lm -o abi_example && LD_LIBRARY_PATH=.. ./abi_example
 */
#include <cuda_runtime.h>
#include <math.h>
#include <stdio.h>
#include <stdlib.h>

#include "progrpo.h"

#define CHECK_PG(call)                                                                  \
  do {                                                                                  \
    int rc_ = (call);                                                                   \
    if (rc_ != PG_OK) {                                                                 \
      fprintf(stderr, "%s -> %s (cuda %d)\n", #call, pg_strerror(rc_), pg_last_cuda_error()); \
      return 1;                                                                         \
    }                                                                                   \
  } while (0)
#define CHECK_CUDA(call)                                                     \
  do {                                                                       \
    cudaError_t e_ = (call);                                                 \
    if (e_ != cudaSuccess) {                                                 \
      fprintf(stderr, "%s -> %s\n", #call, cudaGetErrorString(e_));          \
      return 1;                                                              \
    }                                                                        \
  } while (0)

int main(void) {
  enum { G = 2, N0 = 16, K = 8, D = 4 * 32 * 32, T = 10 };
  const int32_t stage_step[1] = {3}, stage_keep[1] = {K};
  pg_config cfg = {G, N0, D, T, 1, stage_step, stage_keep, 42u, 0, PG_VEL_F32, 1, 1e-6f};
  pg_rollout *h = NULL;
  CHECK_PG(pg_rollout_init(&cfg, &h));

  const int rows = G * N0;
  float *x[2], *vel, *logp, *scores, *rewards, *adv;
  int32_t *keep, *src, *ids;
  CHECK_CUDA(cudaMalloc((void **)&x[0], sizeof(float) * rows * D));
  CHECK_CUDA(cudaMalloc((void **)&x[1], sizeof(float) * rows * D));
  CHECK_CUDA(cudaMalloc((void **)&vel, sizeof(float) * rows * D));
  CHECK_CUDA(cudaMalloc((void **)&logp, sizeof(float) * rows));
  CHECK_CUDA(cudaMalloc((void **)&scores, sizeof(float) * rows));
  CHECK_CUDA(cudaMalloc((void **)&rewards, sizeof(float) * rows));
  CHECK_CUDA(cudaMalloc((void **)&adv, sizeof(float) * rows));
  CHECK_CUDA(cudaMalloc((void **)&keep, sizeof(int32_t) * rows));
  CHECK_CUDA(cudaMalloc((void **)&src, sizeof(int32_t) * rows));
  CHECK_CUDA(cudaMalloc((void **)&ids, sizeof(int32_t) * rows));

  /* x_0 ~ N(0, I): noise stream 1, keyed by the trajectory ids of the fresh handle */
  CHECK_PG(pg_rollout_traj_ids(h, ids, NULL));
  CHECK_PG(pg_normal_rows(cfg.seed, 0, 1, rows, D, ids, x[0], NULL));

  int cur = 0, n_active = rows;
  const double dt = 1.0 / T;
  for (int s = 0; s < T; ++s) {
    /* stand-in for the denoiser: a fresh N(0, 1) prediction for the active rows (noise stream 2) */
    CHECK_PG(pg_rollout_traj_ids(h, ids, NULL));
    CHECK_PG(pg_normal_rows(cfg.seed, s, 2, n_active, D, ids, vel, NULL));
    const int32_t *gather = NULL;
    if (s == stage_step[0]) {
      pg_preview_coef pc = {1.0, 1.0 - s * dt};
      CHECK_PG(pg_score(h, &pc, x[cur], vel, scores, NULL, NULL));
      CHECK_PG(pg_prune_ovf(h, 0, scores, keep, src, NULL, NULL));
      gather = src;
      n_active = G * K;
    }
    pg_step_coef sc = {1.0, dt, 0.7 * sqrt(dt)};
    float *out = gather ? x[cur ^ 1] : x[cur];
    CHECK_PG(pg_step(h, s, &sc, x[cur], vel, gather, out, logp, NULL));
    if (gather) cur ^= 1;
  }
  pg_preview_coef mean_of_x = {1.0, 0.0};
  CHECK_PG(pg_score(h, &mean_of_x, x[cur], NULL, rewards, NULL, NULL));
  CHECK_PG(pg_advantages(h, rewards, adv, NULL, NULL, NULL));

  int32_t active = 0, next = 0, status = 0;
  CHECK_PG(pg_rollout_status(h, &active, &next, &status));
  float host_adv[G * K], host_logp[G * K];
  CHECK_CUDA(cudaMemcpy(host_adv, adv, sizeof host_adv, cudaMemcpyDeviceToHost));
  CHECK_CUDA(cudaMemcpy(host_logp, logp, sizeof host_logp, cudaMemcpyDeviceToHost));
  int ok = (active == G * K && next == T && status == 0);
  for (int g = 0; g < G; ++g) {
    double sum = 0.0;
    printf("group %d advantages:", g);
    for (int i = 0; i < K; ++i) {
      printf(" % .4f", host_adv[g * K + i]);
      sum += host_adv[g * K + i];
    }
    printf("   (sum % .2e, last-step mean log-prob % .4f)\n", sum, host_logp[g * K]);
    if (fabs(sum) > 1e-4) ok = 0;
  }
  printf("%llu kernel launches\n", (unsigned long long)pg_launch_count());
  pg_rollout_destroy(h);
  cudaFree(x[0]); cudaFree(x[1]); cudaFree(vel); cudaFree(logp); cudaFree(scores);
  cudaFree(rewards); cudaFree(adv); cudaFree(keep); cudaFree(src); cudaFree(ids);
  return ok ? 0 : 2;
}
