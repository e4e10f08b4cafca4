// C ABI of the rollout library: handle, schedule cursor, argument checks, and the host-buffer
// end-to-end driver.  All arithmetic is in the kernels of pg_step.cu / pg_score.cu / pg_ovf.cu /
// pg_compact.cu; this file only validates, keeps the cursor and enqueues.
#include "pg_common.cuh"

#include <nvtx3/nvToolsExt.h>

#include <atomic>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

namespace pg {

static std::atomic<uint64_t> g_launches{0};
static thread_local int g_last_cuda_error = 0;

void note_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }
int cuda_fail(cudaError_t e) {
  g_last_cuda_error = (int)e;
  (void)cudaGetLastError();   // clear the sticky-less error so later calls start clean
  return PG_ECUDA;
}

}  // namespace pg

struct pg_rollout {
  pg_config cfg;
  std::vector<int32_t> stage_step, stage_keep;
  int stage_cur = 0;      // stages already pruned
  int next_step = 0;
  int k_cur = 0;          // active trajectories per group
  int k_prev = 0;         // group size before the most recent prune (for pg_compact)
  int device = 0;
  int32_t* d_traj[2] = {nullptr, nullptr};
  int traj_cur = 0;
  float* d_partials = nullptr;
  unsigned int* d_tickets = nullptr;
  int32_t* d_status = nullptr;
  double* d_obj_part = nullptr;        // [1024] per-CTA partial sums of the objective kernel
  unsigned int* d_obj_ticket = nullptr; // its arrival counter, zero between launches
  // streams and events of the host-buffer driver, created on its first use with this handle
  cudaStream_t host_compute = nullptr, host_copy = nullptr;
  cudaEvent_t v_ready[2] = {nullptr, nullptr}, v_free[2] = {nullptr, nullptr};
  long long* d_step_off = nullptr;   // [T + 1] offsets of the steps in a packed per-step row array
  long long total_step_rows = 0;
};

using pg::cuda_fail;

static bool aligned16(const void* p) { return ((uintptr_t)p & 15) == 0; }

// Named range around a library call for timeline tools (NVTX; a no-op costing a pointer test when
// no tool is attached).
struct TraceRange {
  explicit TraceRange(const char* name) { nvtxRangePushA(name); }
  ~TraceRange() { nvtxRangePop(); }
  TraceRange(const TraceRange&) = delete;
  TraceRange& operator=(const TraceRange&) = delete;
};

// A handle's device memory belongs to the device that was current at pg_rollout_init: a call made
// with another device current would hand that device pointers it cannot reach.
static int wrong_device(const pg_rollout* h) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return cuda_fail(cudaGetLastError());
  return dev == h->device ? PG_OK : PG_EDEVICE;
}

static int validate_config(const pg_config* c) {
  if (!c) return PG_EINVAL;
  if (c->n_groups < 1 || c->n_expand < 1 || c->n_expand > PG_MAX_GROUP) return PG_EINVAL;
  if (c->elems < 4 || (c->elems & 3)) return PG_EINVAL;
  if (c->n_steps < 1 || c->n_stages < 0) return PG_EINVAL;
  if (c->n_stages > 0 && (!c->stage_step || !c->stage_keep)) return PG_EINVAL;
  if (c->vel_dtype != PG_VEL_F32 && c->vel_dtype != PG_VEL_BF16) return PG_EINVAL;
  if (!(c->adv_eps >= 0.f)) return PG_EINVAL;
  if (c->group_offset < 0) return PG_EINVAL;
  const long long ids = ((long long)c->group_offset + c->n_groups) * c->n_expand;
  if (ids > 0x7FFFFFFFLL) return PG_EINVAL;
  int prev_step = -1, prev_keep = c->n_expand;
  for (int i = 0; i < c->n_stages; ++i) {
    if (c->stage_step[i] <= prev_step || c->stage_step[i] >= c->n_steps) return PG_EINVAL;
    if (c->stage_keep[i] < 1 || c->stage_keep[i] > prev_keep) return PG_EINVAL;
    prev_step = c->stage_step[i];
    prev_keep = c->stage_keep[i];
  }
  return PG_OK;
}

extern "C" {

int pg_rollout_init(const pg_config* cfg, pg_rollout** out) {
  if (!out) return PG_EINVAL;
  *out = nullptr;
  const int rc = validate_config(cfg);
  if (rc != PG_OK) return rc;
  pg_rollout* h = new (std::nothrow) pg_rollout();
  if (!h) return PG_ENOMEM;
  h->cfg = *cfg;
  h->stage_step.assign(cfg->stage_step, cfg->stage_step + cfg->n_stages);
  h->stage_keep.assign(cfg->stage_keep, cfg->stage_keep + cfg->n_stages);
  h->cfg.stage_step = h->stage_step.data();
  h->cfg.stage_keep = h->stage_keep.data();
  h->k_cur = cfg->n_expand;
  const size_t rows = (size_t)cfg->n_groups * cfg->n_expand;
  // partial-sum slots: the largest need over the row counts this schedule will launch with
  size_t slots = rows * (size_t)pg::row_geometry((long long)rows, cfg->elems).chunks;
  for (int i = 0; i < cfg->n_stages; ++i) {
    const long long r = (long long)cfg->n_groups * cfg->stage_keep[i];
    const size_t need = (size_t)r * (size_t)pg::row_geometry(r, cfg->elems).chunks;
    if (need > slots) slots = need;
  }
  cudaError_t e = cudaGetDevice(&h->device);
  if (e == cudaSuccess) e = cudaMalloc(&h->d_traj[0], rows * sizeof(int32_t));
  if (e == cudaSuccess) e = cudaMalloc(&h->d_traj[1], rows * sizeof(int32_t));
  if (e == cudaSuccess) e = cudaMalloc(&h->d_partials, 2 * slots * sizeof(float))   /* up to two sums per row */;
  if (e == cudaSuccess) e = cudaMalloc(&h->d_tickets, rows * sizeof(unsigned int));
  if (e == cudaSuccess) e = cudaMalloc(&h->d_status, sizeof(int32_t));
  if (e == cudaSuccess) e = cudaMalloc(&h->d_obj_part, 1024 * sizeof(double));
  if (e == cudaSuccess) e = cudaMalloc(&h->d_obj_ticket, sizeof(unsigned int));
  if (e == cudaSuccess) e = cudaMemset(h->d_obj_ticket, 0, sizeof(unsigned int));
  std::vector<long long> step_off((size_t)cfg->n_steps + 1, 0);
  {
    int k = cfg->n_expand, si = 0;
    for (int s = 0; s < cfg->n_steps; ++s) {
      if (si < cfg->n_stages && cfg->stage_step[si] == s) k = cfg->stage_keep[si++];
      step_off[s + 1] = step_off[s] + (long long)cfg->n_groups * k;
    }
  }
  h->total_step_rows = step_off.back();
  if (e == cudaSuccess) e = cudaMalloc(&h->d_step_off, step_off.size() * sizeof(long long));
  if (e == cudaSuccess)
    e = cudaMemcpy(h->d_step_off, step_off.data(), step_off.size() * sizeof(long long), cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMemset(h->d_tickets, 0, rows * sizeof(unsigned int));
  if (e == cudaSuccess) e = cudaMemset(h->d_status, 0, sizeof(int32_t));
  int lrc = PG_OK;
  if (e == cudaSuccess)
    lrc = pg::launch_iota(h->d_traj[0], (int)rows, cfg->group_offset * cfg->n_expand, nullptr);
  if (e == cudaSuccess && lrc == PG_OK) e = cudaStreamSynchronize(nullptr);
  if (e != cudaSuccess || lrc != PG_OK) {
    const int code = (e == cudaErrorMemoryAllocation) ? PG_ENOMEM : (e != cudaSuccess ? cuda_fail(e) : lrc);
    pg_rollout_destroy(h);
    return code;
  }
  *out = h;
  return PG_OK;
}

int pg_rollout_destroy(pg_rollout* h) {
  if (!h) return PG_OK;
  cudaFree(h->d_traj[0]);
  cudaFree(h->d_traj[1]);
  cudaFree(h->d_partials);
  cudaFree(h->d_tickets);
  cudaFree(h->d_status);
  cudaFree(h->d_obj_part);
  cudaFree(h->d_obj_ticket);
  cudaFree(h->d_step_off);
  for (int i = 0; i < 2; ++i) {
    if (h->v_ready[i]) cudaEventDestroy(h->v_ready[i]);
    if (h->v_free[i]) cudaEventDestroy(h->v_free[i]);
  }
  if (h->host_compute) cudaStreamDestroy(h->host_compute);
  if (h->host_copy) cudaStreamDestroy(h->host_copy);
  delete h;
  return PG_OK;
}

int pg_rollout_reset(pg_rollout* h, void* stream) {
  if (!h) return PG_EINVAL;
  if (const int rc_dev = wrong_device(h)) return rc_dev;
  cudaStream_t st = (cudaStream_t)stream;
  const int rows = h->cfg.n_groups * h->cfg.n_expand;
  h->stage_cur = 0;
  h->next_step = 0;
  h->k_cur = h->cfg.n_expand;
  h->k_prev = 0;
  h->traj_cur = 0;
  PG_CUDA(cudaMemsetAsync(h->d_status, 0, sizeof(int32_t), st));
  PG_CUDA(cudaMemsetAsync(h->d_tickets, 0, (size_t)rows * sizeof(unsigned int), st));
  return pg::launch_iota(h->d_traj[0], rows, h->cfg.group_offset * h->cfg.n_expand, st);
}

int pg_rollout_restore(pg_rollout* h, int32_t next_step, int32_t stages_done, const int32_t* traj_ids,
                       void* stream) {
  if (!h || !traj_ids) return PG_EINVAL;
  if (const int rc_dev = wrong_device(h)) return rc_dev;
  if (next_step < 0 || next_step > h->cfg.n_steps || stages_done < 0 || stages_done > h->cfg.n_stages)
    return PG_EINVAL;
  // the cursor must be one the schedule can reach: every stage before next_step is done, and the
  // stage scheduled at next_step itself may or may not have been pruned yet
  for (int i = 0; i < h->cfg.n_stages; ++i) {
    const bool done = i < stages_done;
    if (h->stage_step[i] < next_step && !done) return PG_ESTATE;
    if (h->stage_step[i] > next_step && done) return PG_ESTATE;
  }
  const int k_cur = stages_done > 0 ? h->stage_keep[stages_done - 1] : h->cfg.n_expand;
  const int k_prev = stages_done > 1 ? h->stage_keep[stages_done - 2]
                                     : (stages_done == 1 ? h->cfg.n_expand : 0);
  cudaStream_t st = (cudaStream_t)stream;
  PG_CUDA(cudaMemcpyAsync(h->d_traj[0], traj_ids, (size_t)h->cfg.n_groups * k_cur * sizeof(int32_t),
                          cudaMemcpyDeviceToDevice, st));
  PG_CUDA(cudaMemsetAsync(h->d_status, 0, sizeof(int32_t), st));
  PG_CUDA(cudaMemsetAsync(h->d_tickets, 0,
                          (size_t)h->cfg.n_groups * h->cfg.n_expand * sizeof(unsigned int), st));
  h->traj_cur = 0;
  h->next_step = next_step;
  h->stage_cur = stages_done;
  h->k_cur = k_cur;
  h->k_prev = k_prev;
  return PG_OK;
}

int pg_rollout_status(pg_rollout* h, int32_t* n_active, int32_t* next_step, int32_t* device_status) {
  if (!h) return PG_EINVAL;
  if (const int rc_dev = wrong_device(h)) return rc_dev;
  PG_CUDA(cudaDeviceSynchronize());
  int32_t st = 0;
  PG_CUDA(cudaMemcpy(&st, h->d_status, sizeof(int32_t), cudaMemcpyDeviceToHost));
  if (n_active) *n_active = h->cfg.n_groups * h->k_cur;
  if (next_step) *next_step = h->next_step;
  if (device_status) *device_status = st;
  if (st & 4) return PG_EINDEX;
  if (st & 2) return PG_ETIMEOUT;
  if (st & 1) return PG_ENONFINITE;
  return PG_OK;
}

}  // extern "C"

static int step_impl(pg_rollout* h, int32_t step, const pg_step_coef* coef, const float* x_in,
                     const void* vel, const int32_t* src_rows, float* x_out, float* logp_out,
                     float* xmean_out, void* stream) {
  TraceRange trace_range("pg_step");
  if (!h || !coef || !x_in || !vel || !x_out || !logp_out) return PG_EINVAL;
  if (const int rc_dev = wrong_device(h)) return rc_dev;
  if (!aligned16(x_in) || !aligned16(vel) || !aligned16(x_out)) return PG_EINVAL;
  if (src_rows) {
    // a gathered step reads rows that other CTAs may already have overwritten if the output shares
    // any byte with the input: refuse every overlap, not only x_out == x_in
    const size_t row_bytes = (size_t)h->cfg.elems * sizeof(float);
    const uintptr_t in_lo = (uintptr_t)x_in, out_lo = (uintptr_t)x_out;
    const uintptr_t in_hi = in_lo + (size_t)h->cfg.n_groups * (h->k_prev > 0 ? h->k_prev : h->k_cur) * row_bytes;
    const uintptr_t out_hi = out_lo + (size_t)h->cfg.n_groups * h->k_cur * row_bytes;
    if (in_lo < out_hi && out_lo < in_hi) return PG_EINVAL;
  }
  if (!(coef->noise_std >= 0.0) || !std::isfinite(coef->c_x) || !std::isfinite(coef->c_v) ||
      !std::isfinite(coef->noise_std))
    return PG_EINVAL;
  if (step != h->next_step || step >= h->cfg.n_steps) return PG_ESTATE;
  if (h->stage_cur < h->cfg.n_stages && h->stage_step[h->stage_cur] == step) return PG_ESTATE;
  const int rows = h->cfg.n_groups * h->k_cur;
  pg::RowScratch scratch{h->d_partials, h->d_tickets};
  const int rc = pg::launch_step(rows, h->cfg.elems, h->cfg.vel_dtype, x_in, vel, src_rows,
                                 h->d_traj[h->traj_cur], x_out, logp_out, h->cfg.seed, step,
                                 coef->c_x, coef->c_v, coef->noise_std, h->cfg.logp_mean, scratch,
                                 (cudaStream_t)stream,
                                 src_rows ? h->cfg.n_groups * h->k_prev : rows, h->d_status, xmean_out);
  if (rc == PG_OK) h->next_step = step + 1;
  return rc;
}

extern "C" {

int pg_step(pg_rollout* h, int32_t step, const pg_step_coef* coef, const float* x_in,
            const void* vel, const int32_t* src_rows, float* x_out, float* logp_out, void* stream) {
  return step_impl(h, step, coef, x_in, vel, src_rows, x_out, logp_out, nullptr, stream);
}

int pg_step_reward(pg_rollout* h, int32_t step, const pg_step_coef* coef, const float* x_in,
                   const void* vel, const int32_t* src_rows, float* x_out, float* logp_out,
                   float* reward_out, void* stream) {
  if (!reward_out) return PG_EINVAL;
  return step_impl(h, step, coef, x_in, vel, src_rows, x_out, logp_out, reward_out, stream);
}

int pg_score_preview(pg_rollout* h, const pg_preview_coef* coef, const float* x, const void* vel,
                     float* scores_out, void* preview_out, int32_t preview_dtype, void* stream) {
  TraceRange trace_range("pg_score");
  if (!h || !coef || !x || !scores_out) return PG_EINVAL;
  if (const int rc_dev = wrong_device(h)) return rc_dev;
  if (!std::isfinite(coef->p_x) || !std::isfinite(coef->p_v)) return PG_EINVAL;
  if (coef->p_v != 0.0 && !vel) return PG_EINVAL;
  if (preview_out && preview_dtype != PG_VEL_F32 && preview_dtype != PG_VEL_BF16) return PG_EINVAL;
  if (!aligned16(x) || !aligned16(vel) || !aligned16(preview_out)) return PG_EINVAL;
  const int rows = h->cfg.n_groups * h->k_cur;
  pg::RowScratch scratch{h->d_partials, h->d_tickets};
  return pg::launch_score(rows, h->cfg.elems, h->cfg.vel_dtype, x, vel, coef->p_x, coef->p_v,
                          scores_out, preview_out, preview_dtype == PG_VEL_BF16, scratch,
                          (cudaStream_t)stream);
}

int pg_score(pg_rollout* h, const pg_preview_coef* coef, const float* x, const void* vel,
             float* scores_out, float* preview_out, void* stream) {
  return pg_score_preview(h, coef, x, vel, scores_out, preview_out, PG_VEL_F32, stream);
}

int pg_preview(pg_rollout* h, const pg_preview_coef* coef, const float* x, const void* vel, void* out,
               int32_t out_dtype, void* stream) {
  TraceRange trace_range("pg_preview");
  if (!h || !coef || !x || !vel || !out) return PG_EINVAL;
  if (const int rc_dev = wrong_device(h)) return rc_dev;
  if (out_dtype != PG_VEL_F32 && out_dtype != PG_VEL_BF16) return PG_EINVAL;
  if (!std::isfinite(coef->p_x) || !std::isfinite(coef->p_v)) return PG_EINVAL;
  if (!aligned16(x) || !aligned16(vel) || !aligned16(out)) return PG_EINVAL;
  return pg::launch_preview(h->cfg.n_groups * h->k_cur, h->cfg.elems, h->cfg.vel_dtype, x, vel, coef->p_x,
                            coef->p_v, out, out_dtype == PG_VEL_BF16, (cudaStream_t)stream);
}

int pg_prune_ovf(pg_rollout* h, int32_t stage, const float* scores, int32_t* keep_idx,
                 int32_t* src_rows, float* sel_var, void* stream) {
  TraceRange trace_range("pg_prune_ovf");
  if (!h || !scores || !keep_idx) return PG_EINVAL;
  if (const int rc_dev = wrong_device(h)) return rc_dev;
  if (stage != h->stage_cur || stage >= h->cfg.n_stages) return PG_ESTATE;
  if (h->stage_step[stage] != h->next_step) return PG_ESTATE;
  const int n = h->k_cur, k = h->stage_keep[stage];
  const int rc = pg::launch_ovf(h->cfg.n_groups, n, k, scores, keep_idx, src_rows, sel_var, nullptr,
                                nullptr, 0.f, h->d_traj[h->traj_cur], h->d_traj[h->traj_cur ^ 1],
                                h->d_status, (cudaStream_t)stream);
  if (rc != PG_OK) return rc;
  h->traj_cur ^= 1;
  h->k_prev = n;
  h->k_cur = k;
  h->stage_cur = stage + 1;
  return PG_OK;
}

int pg_prune_uniform(pg_rollout* h, int32_t stage, int32_t* keep_idx, int32_t* src_rows, void* stream) {
  TraceRange trace_range("pg_prune_uniform");
  if (!h || !keep_idx) return PG_EINVAL;
  if (const int rc_dev = wrong_device(h)) return rc_dev;
  if (stage != h->stage_cur || stage >= h->cfg.n_stages) return PG_ESTATE;
  if (h->stage_step[stage] != h->next_step) return PG_ESTATE;
  const int n = h->k_cur, k = h->stage_keep[stage];
  const int rc = pg::launch_uniform_select(h->cfg.n_groups, n, k, h->cfg.seed, (uint32_t)stage,
                                           (uint32_t)h->cfg.group_offset, keep_idx, src_rows,
                                           h->d_traj[h->traj_cur], h->d_traj[h->traj_cur ^ 1],
                                           (cudaStream_t)stream);
  if (rc != PG_OK) return rc;
  h->traj_cur ^= 1;
  h->k_prev = n;
  h->k_cur = k;
  h->stage_cur = stage + 1;
  return PG_OK;
}

int pg_group_stats(int32_t n_groups, int32_t n, const float* scores, float delta, float* mean,
                   float* std, float* clustered_frac, void* stream) {
  if (n_groups < 0 || n < 1 || !(delta >= 0.f)) return PG_EINVAL;
  if (n_groups == 0) return PG_OK;
  if (!scores) return PG_EINVAL;
  return pg::launch_group_stats(n_groups, n, scores, (double)delta, mean, std, clustered_frac,
                                (cudaStream_t)stream);
}

int pg_compact(pg_rollout* h, const int32_t* keep_idx, const void* src, void* dst, size_t row_bytes,
               void* stream) {
  TraceRange trace_range("pg_compact");
  if (!h || !keep_idx || !src || !dst || row_bytes == 0) return PG_EINVAL;
  if (const int rc_dev = wrong_device(h)) return rc_dev;
  if (h->k_prev == 0) return PG_ESTATE;
  const size_t src_bytes = (size_t)h->cfg.n_groups * h->k_prev * row_bytes;
  const size_t dst_bytes = (size_t)h->cfg.n_groups * h->k_cur * row_bytes;
  const uintptr_t s = (uintptr_t)src, d = (uintptr_t)dst;
  if (s < d + dst_bytes && d < s + src_bytes) return PG_EINVAL;   // overlap
  return pg::launch_compact(h->cfg.n_groups, h->k_prev, h->k_cur, keep_idx, src, dst, row_bytes,
                            (cudaStream_t)stream, h->d_status);
}

int pg_advantages(pg_rollout* h, const float* rewards, float* adv, float* mean, float* std,
                  void* stream) {
  TraceRange trace_range("pg_advantages");
  if (!h || !rewards || !adv) return PG_EINVAL;
  if (const int rc_dev = wrong_device(h)) return rc_dev;
  return pg::launch_advantages(h->cfg.n_groups, h->k_cur, rewards, h->cfg.adv_eps, adv, mean, std,
                               (cudaStream_t)stream);
}

int pg_policy_logprob(pg_rollout* h, const pg_step_coef* coef, const float* x, const float* x_next,
                      const void* vel, const void* vel_ref, float* logp_out, float* kl_out, void* stream) {
  TraceRange trace_range("pg_policy_logprob");
  if (!h || !coef || !x || !x_next || !vel || !logp_out) return PG_EINVAL;
  if (const int rc_dev = wrong_device(h)) return rc_dev;
  if ((vel_ref == nullptr) != (kl_out == nullptr)) return PG_EINVAL;
  if (!aligned16(x) || !aligned16(x_next) || !aligned16(vel) || !aligned16(vel_ref)) return PG_EINVAL;
  if (!(coef->noise_std > 0.0) || !std::isfinite(coef->c_x) || !std::isfinite(coef->c_v) ||
      !std::isfinite(coef->noise_std))
    return PG_EINVAL;
  pg::RowScratch scratch{h->d_partials, h->d_tickets};
  return pg::launch_policy_logprob(h->cfg.n_groups * h->k_cur, h->cfg.elems, h->cfg.vel_dtype, x, x_next,
                                   vel, vel_ref, coef->c_x, coef->c_v, coef->noise_std,
                                   h->cfg.logp_mean, logp_out, kl_out, scratch, (cudaStream_t)stream);
}

int pg_policy_objective(pg_rollout* h, int32_t n_steps, const float* logp_new, const float* logp_old,
                        const float* kl, const float* adv, float clip_eps, float beta, float* ratio,
                        float* dlogp, float* objective, void* stream) {
  TraceRange trace_range("pg_policy_objective");
  if (!h || n_steps < 1 || !logp_new || !logp_old || !adv || !dlogp || !objective) return PG_EINVAL;
  if (const int rc_dev = wrong_device(h)) return rc_dev;
  if (!(clip_eps >= 0.f) || !std::isfinite(beta)) return PG_EINVAL;
  return pg::launch_policy_objective(n_steps, h->cfg.n_groups * h->k_cur, logp_new, logp_old, kl, adv,
                                     clip_eps, beta, ratio, dlogp, objective, h->d_obj_part, h->d_obj_ticket,
                                     (cudaStream_t)stream);
}

int pg_policy_backward(pg_rollout* h, const pg_step_coef* coef, const float* x, const float* x_next,
                       const void* vel, const void* vel_ref, const float* dlogp, double dkl,
                       void* grad_vel, void* stream) {
  TraceRange trace_range("pg_policy_backward");
  if (!h || !coef || !x || !x_next || !vel || !dlogp || !grad_vel) return PG_EINVAL;
  if (const int rc_dev = wrong_device(h)) return rc_dev;
  if (!aligned16(x) || !aligned16(x_next) || !aligned16(vel) || !aligned16(vel_ref) ||
      !aligned16(grad_vel))
    return PG_EINVAL;
  if (!(coef->noise_std > 0.0) || !std::isfinite(coef->c_x) || !std::isfinite(coef->c_v) ||
      !std::isfinite(coef->noise_std) || !std::isfinite(dkl))
    return PG_EINVAL;
  return pg::launch_policy_backward(h->cfg.n_groups * h->k_cur, h->cfg.elems, h->cfg.vel_dtype, x, x_next,
                                    vel, vel_ref, coef->c_x, coef->c_v, coef->noise_std,
                                    h->cfg.logp_mean, dlogp, dkl, grad_vel, (cudaStream_t)stream);
}

int pg_ovf_select_batched(int32_t n_groups, int32_t n, int32_t k, const float* scores,
                          int32_t* keep_idx, float* kept_scores, float* adv, float adv_eps,
                          int32_t* status, void* stream) {
  TraceRange trace_range("pg_ovf_select_batched");
  if (n_groups < 0 || n < 1 || n > PG_MAX_GROUP || k < 1 || k > n) return PG_EINVAL;
  if (!(adv_eps >= 0.f)) return PG_EINVAL;
  if (n_groups == 0) return PG_OK;
  if (!scores || !keep_idx) return PG_EINVAL;
  return pg::launch_ovf(n_groups, n, k, scores, keep_idx, nullptr, nullptr, kept_scores, adv,
                        adv_eps, nullptr, nullptr, status, (cudaStream_t)stream);
}

int pg_rollout_traj_ids(pg_rollout* h, int32_t* dst, void* stream) {
  if (!h || !dst) return PG_EINVAL;
  if (const int rc_dev = wrong_device(h)) return rc_dev;
  PG_CUDA(cudaMemcpyAsync(dst, h->d_traj[h->traj_cur],
                          (size_t)h->cfg.n_groups * h->k_cur * sizeof(int32_t),
                          cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
  return PG_OK;
}

int pg_survivor_rows(pg_rollout* h, const int32_t* keep_idx_packed, int32_t* rows_out, void* stream) {
  TraceRange trace_range("pg_survivor_rows");
  if (!h || !rows_out) return PG_EINVAL;
  if (const int rc_dev = wrong_device(h)) return rc_dev;
  if (h->cfg.n_stages > 0 && !keep_idx_packed) return PG_EINVAL;
  return pg::launch_survivor_rows(h->cfg.n_groups, h->cfg.n_expand, h->cfg.n_steps, h->cfg.n_stages,
                                  h->stage_step.data(), h->stage_keep.data(), keep_idx_packed, rows_out,
                                  h->d_status, (cudaStream_t)stream);
}

int pg_survivor_logp(pg_rollout* h, const int32_t* rows, const float* logp_packed, float* logp_out,
                     void* stream) {
  TraceRange trace_range("pg_survivor_logp");
  if (!h || !rows || !logp_packed || !logp_out) return PG_EINVAL;
  if (const int rc_dev = wrong_device(h)) return rc_dev;
  const int k_final = h->cfg.n_stages > 0 ? h->stage_keep.back() : h->cfg.n_expand;
  return pg::launch_survivor_logp(rows, logp_packed, logp_out, h->d_step_off, h->cfg.n_steps,
                                  h->cfg.n_groups * k_final, h->d_status, (cudaStream_t)stream);
}

int pg_gather_rows(pg_rollout* h, const int32_t* rows, int32_t n_out, int32_t n_in, const void* src,
                   void* dst, size_t row_bytes, void* stream) {
  TraceRange trace_range("pg_gather_rows");
  if (!h || n_out < 0 || n_in < 0 || row_bytes == 0) return PG_EINVAL;
  if (const int rc_dev = wrong_device(h)) return rc_dev;
  if (n_out == 0) return PG_OK;
  if (!rows || !src || !dst || n_in == 0) return PG_EINVAL;
  const uintptr_t s = (uintptr_t)src, d = (uintptr_t)dst;
  if (s < d + (size_t)n_out * row_bytes && d < s + (size_t)n_in * row_bytes) return PG_EINVAL;   // overlap
  // one "group" of n_in rows from which n_out are taken: the compaction kernel's gather
  return pg::launch_compact(1, n_in, n_out, rows, src, dst, row_bytes, (cudaStream_t)stream, h->d_status);
}

int pg_selftest_bounded_wait(pg_rollout* h, void* stream) {
  if (!h) return PG_EINVAL;
  if (const int rc_dev = wrong_device(h)) return rc_dev;
  return pg::launch_wait_selftest(h->d_status, (cudaStream_t)stream);
}

int pg_philox_raw(int64_t n, const uint32_t* ctr, const uint32_t* key, uint32_t* out, void* stream) {
  if (n < 0 || (n > 0 && (!ctr || !key || !out)) || !aligned16(out)) return PG_EINVAL;
  return pg::launch_philox_raw(n, ctr, key, out, (cudaStream_t)stream);
}

int pg_normal_rows(uint64_t seed, int32_t step, int32_t stream_id, int32_t n_rows, int32_t d,
                   const int32_t* traj_id, float* out, void* stream) {
  if (n_rows < 0 || d < 4 || (d & 3) || step < 0 || stream_id < 0) return PG_EINVAL;
  if (n_rows > 0 && (!traj_id || !out || !aligned16(out))) return PG_EINVAL;
  return pg::launch_normal_rows(seed, step, stream_id, n_rows, d, traj_id, out, (cudaStream_t)stream);
}

const char* pg_strerror(int code) {
  switch (code) {
    case PG_OK: return "ok";
    case PG_EINVAL: return "invalid argument (null pointer, shape, alignment or overlap)";
    case PG_ESTATE: return "call out of sequence for the rollout schedule";
    case PG_ECUDA: return "CUDA runtime error (see pg_last_cuda_error)";
    case PG_ENONFINITE: return "non-finite scores were seen by the selection";
    case PG_ETIMEOUT: return "a bounded device-side wait expired";
    case PG_ENOMEM: return "out of memory";
    case PG_EINDEX: return "a gather index (src_rows / keep_idx) was out of range; the rows were not read";
    case PG_ECAPACITY: return "request exceeds the capacity of a fixed built-in buffer";
    case PG_EDEVICE: return "the handle belongs to another device than the current one";
    default: return "unknown error code";
  }
}

int pg_last_cuda_error(void) { return pg::g_last_cuda_error; }
uint64_t pg_launch_count(void) { return pg::g_launches.load(std::memory_order_relaxed); }

// ---------------------------------------------------------------- host-buffer driver

static size_t round256(size_t b) { return (b + 255) & ~(size_t)255; }

struct HostPlan {
  size_t rows0, vel_elem, x_bytes, v_bytes, total_logp, total_keep;
  size_t off_x[2], off_v[2], off_scores, off_keep, off_src, off_logp, off_rewards, off_adv,
      off_traj, total;
};

static HostPlan make_plan(const pg_config* c) {
  HostPlan p;
  p.rows0 = (size_t)c->n_groups * c->n_expand;
  p.vel_elem = c->vel_dtype == PG_VEL_BF16 ? 2 : 4;
  p.x_bytes = p.rows0 * c->elems * sizeof(float);
  p.v_bytes = p.rows0 * c->elems * p.vel_elem;
  p.total_logp = 0;
  p.total_keep = 0;
  int k = c->n_expand, si = 0;
  for (int s = 0; s < c->n_steps; ++s) {
    if (si < c->n_stages && c->stage_step[si] == s) {
      k = c->stage_keep[si++];
      p.total_keep += (size_t)c->n_groups * k;
    }
    p.total_logp += (size_t)c->n_groups * k;
  }
  size_t o = 0;
  for (int i = 0; i < 2; ++i) { p.off_x[i] = o; o += round256(p.x_bytes); }
  for (int i = 0; i < 2; ++i) { p.off_v[i] = o; o += round256(p.v_bytes); }
  p.off_scores = o;  o += round256(p.rows0 * 4);
  p.off_keep = o;    o += round256((p.total_keep + 1) * 4);
  p.off_src = o;     o += round256(p.rows0 * 4);
  p.off_logp = o;    o += round256(p.total_logp * 4);
  p.off_rewards = o; o += round256(p.rows0 * 4);
  p.off_adv = o;     o += round256(p.rows0 * 4);
  p.off_traj = o;    o += round256(p.rows0 * 4);
  p.total = o;
  return p;
}

size_t pg_rollout_host_workspace_bytes(const pg_config* cfg) {
  if (validate_config(cfg) != PG_OK) return 0;
  return make_plan(cfg).total;
}

// Streams and events of the host-buffer driver live in the handle: made once, reused by every call.
static int ensure_host_resources(pg_rollout* h) {
  if (!h->host_compute) PG_CUDA(cudaStreamCreateWithFlags(&h->host_compute, cudaStreamNonBlocking));
  if (!h->host_copy) PG_CUDA(cudaStreamCreateWithFlags(&h->host_copy, cudaStreamNonBlocking));
  for (int i = 0; i < 2; ++i) {
    if (!h->v_ready[i]) PG_CUDA(cudaEventCreateWithFlags(&h->v_ready[i], cudaEventDisableTiming));
    if (!h->v_free[i]) PG_CUDA(cudaEventCreateWithFlags(&h->v_free[i], cudaEventDisableTiming));
  }
  return PG_OK;
}

int pg_rollout_host_on(pg_rollout* h, const pg_step_coef* step_coef,
                       const pg_preview_coef* preview_coef, const float* x0,
                       const void* const* vel_steps, const float* const* stage_scores,
                       const float* final_rewards, float* x_final, float* logp, int32_t* keep_idx,
                       float* adv, int32_t* traj_id, void* workspace, size_t workspace_bytes) {
  TraceRange trace_range("pg_rollout_host");
  if (!h) return PG_EINVAL;
  if (const int rc_dev = wrong_device(h)) return rc_dev;
  const pg_config* cfg = &h->cfg;
  if (!step_coef || !vel_steps || !workspace || !aligned16(workspace)) return PG_EINVAL;
  if (cfg->n_stages > 0 && !preview_coef && !stage_scores) return PG_EINVAL;
  const HostPlan pl = make_plan(cfg);
  if (workspace_bytes < pl.total) return PG_EINVAL;
  for (int s = 0; s < cfg->n_steps; ++s)
    if (!vel_steps[s]) return PG_EINVAL;
  for (int i = 0; i < cfg->n_stages; ++i)
    if (!(stage_scores && stage_scores[i]) && !preview_coef) return PG_EINVAL;
  int rc = ensure_host_resources(h);
  if (rc != PG_OK) return rc;

  unsigned char* ws = (unsigned char*)workspace;
  float* d_x[2] = {(float*)(ws + pl.off_x[0]), (float*)(ws + pl.off_x[1])};
  void* d_v[2] = {ws + pl.off_v[0], ws + pl.off_v[1]};
  float* d_scores = (float*)(ws + pl.off_scores);
  int32_t* d_keep = (int32_t*)(ws + pl.off_keep);
  int32_t* d_src = (int32_t*)(ws + pl.off_src);
  float* d_logp = (float*)(ws + pl.off_logp);
  float* d_rewards = (float*)(ws + pl.off_rewards);
  float* d_adv = (float*)(ws + pl.off_adv);
  int32_t* d_traj = (int32_t*)(ws + pl.off_traj);
  cudaStream_t compute = h->host_compute, copy = h->host_copy;
  cudaEvent_t* v_ready = h->v_ready;
  cudaEvent_t* v_free = h->v_free;
  // on an error the streams are drained so that nothing of this call is still in flight
  auto fail = [&](int code) {
    cudaStreamSynchronize(copy);
    cudaStreamSynchronize(compute);
    return code;
  };
#define PG_TRY_CUDA(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) return fail(cuda_fail(e_)); } while (0)
#define PG_TRY(call) do { int r_ = (call); if (r_ != PG_OK) return fail(r_); } while (0)
  PG_TRY(pg_rollout_reset(h, compute));

  // rows alive when the prediction of step s is made
  std::vector<int> rows_pred(cfg->n_steps);
  {
    int k = cfg->n_expand, si = 0;
    for (int s = 0; s < cfg->n_steps; ++s) {
      rows_pred[s] = cfg->n_groups * k;
      if (si < cfg->n_stages && cfg->stage_step[si] == s) k = cfg->stage_keep[si++];
    }
  }
  auto prefetch = [&](int s) -> cudaError_t {
    const int b = s & 1;
    cudaError_t e = cudaSuccess;
    if (s >= 2) e = cudaStreamWaitEvent(copy, v_free[b], 0);
    if (e == cudaSuccess)
      e = cudaMemcpyAsync(d_v[b], vel_steps[s], (size_t)rows_pred[s] * cfg->elems * pl.vel_elem,
                          cudaMemcpyHostToDevice, copy);
    if (e == cudaSuccess) e = cudaEventRecord(v_ready[b], copy);
    return e;
  };

  if (x0) {
    PG_TRY_CUDA(cudaMemcpyAsync(d_x[0], x0, pl.x_bytes, cudaMemcpyHostToDevice, compute));
  } else {
    // initial latents drawn on the device (noise stream 1, keyed by trajectory id): nothing to copy
    PG_TRY(pg::launch_normal_rows(cfg->seed, 0, 1, (int)pl.rows0, cfg->elems, h->d_traj[h->traj_cur],
                                  d_x[0], compute));
  }
  PG_TRY_CUDA(prefetch(0));
  int cur = 0, stage = 0;
  size_t logp_off = 0, keep_off = 0;
  for (int s = 0; s < cfg->n_steps; ++s) {
    if (s + 1 < cfg->n_steps) PG_TRY_CUDA(prefetch(s + 1));
    const int b = s & 1;
    PG_TRY_CUDA(cudaStreamWaitEvent(compute, v_ready[b], 0));
    const int32_t* src = nullptr;
    if (stage < cfg->n_stages && cfg->stage_step[stage] == s) {
      const int rows = cfg->n_groups * h->k_cur;
      if (stage_scores && stage_scores[stage]) {
        PG_TRY_CUDA(cudaMemcpyAsync(d_scores, stage_scores[stage], (size_t)rows * 4,
                                    cudaMemcpyHostToDevice, compute));
      } else {
        PG_TRY(pg_score(h, &preview_coef[stage], d_x[cur], d_v[b], d_scores, nullptr, compute));
      }
      PG_TRY(pg_prune_ovf(h, stage, d_scores, d_keep + keep_off, d_src, nullptr, compute));
      keep_off += (size_t)cfg->n_groups * h->k_cur;
      src = d_src;
      ++stage;
    }
    float* x_out = src ? d_x[cur ^ 1] : d_x[cur];
    if (s == cfg->n_steps - 1 && !final_rewards)      // the last step also reduces the reward stand-in
      PG_TRY(pg_step_reward(h, s, &step_coef[s], d_x[cur], d_v[b], src, x_out, d_logp + logp_off, d_rewards, compute));
    else
      PG_TRY(pg_step(h, s, &step_coef[s], d_x[cur], d_v[b], src, x_out, d_logp + logp_off, compute));
    if (src) cur ^= 1;
    logp_off += (size_t)cfg->n_groups * h->k_cur;
    PG_TRY_CUDA(cudaEventRecord(v_free[b], compute));
  }
  const size_t rows_final = (size_t)cfg->n_groups * h->k_cur;
  if (final_rewards)
    PG_TRY_CUDA(cudaMemcpyAsync(d_rewards, final_rewards, rows_final * 4, cudaMemcpyHostToDevice, compute));
  PG_TRY(pg_advantages(h, d_rewards, d_adv, nullptr, nullptr, compute));
  PG_TRY(pg_rollout_traj_ids(h, d_traj, compute));
  if (x_final) PG_TRY_CUDA(cudaMemcpyAsync(x_final, d_x[cur], rows_final * cfg->elems * 4, cudaMemcpyDeviceToHost, compute));
  if (logp) PG_TRY_CUDA(cudaMemcpyAsync(logp, d_logp, pl.total_logp * 4, cudaMemcpyDeviceToHost, compute));
  if (keep_idx && pl.total_keep) PG_TRY_CUDA(cudaMemcpyAsync(keep_idx, d_keep, pl.total_keep * 4, cudaMemcpyDeviceToHost, compute));
  if (adv) PG_TRY_CUDA(cudaMemcpyAsync(adv, d_adv, rows_final * 4, cudaMemcpyDeviceToHost, compute));
  if (traj_id) PG_TRY_CUDA(cudaMemcpyAsync(traj_id, d_traj, rows_final * 4, cudaMemcpyDeviceToHost, compute));
  int32_t st = 0;
  PG_TRY_CUDA(cudaMemcpyAsync(&st, h->d_status, sizeof(int32_t), cudaMemcpyDeviceToHost, compute));
  PG_TRY_CUDA(cudaStreamSynchronize(compute));
  PG_TRY_CUDA(cudaStreamSynchronize(copy));
  return (st & 4) ? PG_EINDEX : (st & 2) ? PG_ETIMEOUT : (st & 1) ? PG_ENONFINITE : PG_OK;
#undef PG_TRY
#undef PG_TRY_CUDA
}

int pg_rollout_host(const pg_config* cfg, const pg_step_coef* step_coef,
                    const pg_preview_coef* preview_coef, const float* x0,
                    const void* const* vel_steps, const float* const* stage_scores,
                    const float* final_rewards, float* x_final, float* logp, int32_t* keep_idx,
                    float* adv, int32_t* traj_id, void* workspace, size_t workspace_bytes) {
  pg_rollout* h = nullptr;
  int rc = pg_rollout_init(cfg, &h);
  if (rc != PG_OK) return rc;
  rc = pg_rollout_host_on(h, step_coef, preview_coef, x0, vel_steps, stage_scores, final_rewards, x_final,
                          logp, keep_idx, adv, traj_id, workspace, workspace_bytes);
  cudaDeviceSynchronize();
  pg_rollout_destroy(h);
  return rc;
}

// ---------------------------------------------------------------- device-resident driver

struct RunPlan {
  size_t rows0, x_bytes, total_logp, total_keep;
  size_t off_x[2], off_scores, off_keep, off_src, off_logp, off_rewards, off_adv, off_traj, total;
};

static RunPlan make_run_plan(const pg_config* c) {
  RunPlan p;
  const HostPlan hp = make_plan(c);
  p.rows0 = hp.rows0;
  p.x_bytes = hp.x_bytes;
  p.total_logp = hp.total_logp;
  p.total_keep = hp.total_keep;
  size_t o = 0;
  for (int i = 0; i < 2; ++i) { p.off_x[i] = o; o += round256(p.x_bytes); }
  p.off_scores = o;  o += round256(p.rows0 * 4);
  p.off_keep = o;    o += round256((p.total_keep + 1) * 4);
  p.off_src = o;     o += round256(p.rows0 * 4);
  p.off_logp = o;    o += round256(p.total_logp * 4);
  p.off_rewards = o; o += round256(p.rows0 * 4);
  p.off_adv = o;     o += round256(p.rows0 * 4);
  p.off_traj = o;    o += round256(p.rows0 * 4);
  p.total = o;
  return p;
}

size_t pg_rollout_run_workspace_bytes(const pg_config* cfg) {
  if (validate_config(cfg) != PG_OK) return 0;
  return make_run_plan(cfg).total;
}

int pg_rollout_run(pg_rollout* h, const pg_step_coef* step_coef, const pg_preview_coef* preview_coef,
                   const float* x0, const void* const* vel_steps, const float* const* stage_scores,
                   const float* final_rewards, void* workspace, size_t workspace_bytes,
                   pg_rollout_outputs* out, void* stream) {
  TraceRange trace_range("pg_rollout_run");
  if (!h || !step_coef || !x0 || !vel_steps || !workspace || !out || !aligned16(workspace) ||
      !aligned16(x0))
    return PG_EINVAL;
  if (const int rc_dev = wrong_device(h)) return rc_dev;
  const pg_config* cfg = &h->cfg;
  const RunPlan pl = make_run_plan(cfg);
  if (workspace_bytes < pl.total) return PG_EINVAL;
  for (int s = 0; s < cfg->n_steps; ++s)
    if (!vel_steps[s]) return PG_EINVAL;
  for (int i = 0; i < cfg->n_stages; ++i)
    if (!(stage_scores && stage_scores[i]) && !preview_coef) return PG_EINVAL;
  unsigned char* ws = (unsigned char*)workspace;
  float* d_x[2] = {(float*)(ws + pl.off_x[0]), (float*)(ws + pl.off_x[1])};
  float* d_scores = (float*)(ws + pl.off_scores);
  int32_t* d_keep = (int32_t*)(ws + pl.off_keep);
  int32_t* d_src = (int32_t*)(ws + pl.off_src);
  float* d_logp = (float*)(ws + pl.off_logp);
  float* d_rewards = (float*)(ws + pl.off_rewards);
  float* d_adv = (float*)(ws + pl.off_adv);
  int32_t* d_traj = (int32_t*)(ws + pl.off_traj);

  int rc = pg_rollout_reset(h, stream);
  if (rc != PG_OK) return rc;
  const float* x_cur = x0;       // read-only until the first step has written into the workspace
  int cur = -1, stage = 0;       // cur: which workspace half holds x (-1: still x0)
  size_t logp_off = 0, keep_off = 0;
  for (int s = 0; s < cfg->n_steps; ++s) {
    const int32_t* src = nullptr;
    if (stage < cfg->n_stages && cfg->stage_step[stage] == s) {
      const float* sc = (stage_scores && stage_scores[stage]) ? stage_scores[stage] : nullptr;
      if (!sc) {
        rc = pg_score(h, &preview_coef[stage], x_cur, vel_steps[s], d_scores, nullptr, stream);
        if (rc != PG_OK) return rc;
        sc = d_scores;
      }
      rc = pg_prune_ovf(h, stage, sc, d_keep + keep_off, d_src, nullptr, stream);
      if (rc != PG_OK) return rc;
      keep_off += (size_t)cfg->n_groups * h->k_cur;
      src = d_src;
      ++stage;
    }
    float* x_out;
    if (cur < 0) { x_out = d_x[0]; }
    else if (src) { x_out = d_x[cur ^ 1]; }
    else { x_out = d_x[cur]; }
    if (s == cfg->n_steps - 1 && !final_rewards)      // the last step also reduces the reward stand-in
      rc = pg_step_reward(h, s, &step_coef[s], x_cur, vel_steps[s], src, x_out, d_logp + logp_off, d_rewards, stream);
    else
      rc = pg_step(h, s, &step_coef[s], x_cur, vel_steps[s], src, x_out, d_logp + logp_off, stream);
    if (rc != PG_OK) return rc;
    if (cur < 0) cur = 0; else if (src) cur ^= 1;
    x_cur = d_x[cur];
    logp_off += (size_t)cfg->n_groups * h->k_cur;
  }
  const float* rw = final_rewards ? final_rewards : d_rewards;
  rc = pg_advantages(h, rw, d_adv, nullptr, nullptr, stream);
  if (rc != PG_OK) return rc;
  rc = pg_rollout_traj_ids(h, d_traj, stream);
  if (rc != PG_OK) return rc;
  out->x_final = d_x[cur];
  out->logp = d_logp;
  out->keep_idx = d_keep;
  out->adv = d_adv;
  out->rewards = rw;
  out->traj_id = d_traj;
  out->n_final = cfg->n_groups * h->k_cur;
  out->n_logp = (int64_t)pl.total_logp;
  out->n_keep = (int64_t)pl.total_keep;
  return PG_OK;
}

}  // extern "C"
