/*
 * progrpo.h - C ABI of the B200 (sm_100a) hot path of the Pro-GRPO
 * Expand-and-Prune rollout.
 *
 * The library advances G prompt groups of N0 expanded trajectories in lockstep
 * through a T-step reverse-time SDE, scores and prunes them at the scheduled
 * checkpoints with Optimal Variance Filtering (OVF), keeps only survivors in
 * later steps and finally normalises the survivors' rewards into
 * group-relative advantages.  The denoiser, VAE decoder and reward model are
 * outside: their outputs are passed in as tensors.
 *
 * Conventions
 *  - Every function returns 0 (PG_OK) or a negative PG_E* code; nothing aborts
 *    or throws.  pg_strerror() names a code; pg_last_cuda_error() returns the
 *    cudaError_t behind the last PG_ECUDA of the calling thread.
 *  - All tensor pointers are DEVICE pointers owned by the caller, row-major and
 *    contiguous, 16-byte aligned unless stated otherwise.  The library owns
 *    only the opaque handle and its small device scratch (trajectory-id map,
 *    reduction partials, tickets, status word), all released by
 *    pg_rollout_destroy().  pg_config and the coefficient structs are HOST
 *    memory, read during the call only.
 *  - A handle belongs to the device that was current when pg_rollout_init created it; every
 *    call on it must be made with that device current (else PG_EDEVICE, nothing is launched).
 *  - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Calls
 *    enqueue work and return; none synchronises, except pg_rollout_status()
 *    and pg_rollout_host().  All calls on one handle must be issued on one
 *    stream (or be ordered by the caller): the handle's device state is
 *    updated in stream order.
 *  - Rows: at any time the n_active = G * K_i live trajectories are the rows
 *    of the latent tensor, group-major (row = g * K_i + slot).  Step indices
 *    are 0-based.  A stage (s, k) prunes every group to k survivors BEFORE the
 *    SDE update of step s, using the prediction made at x_s; pruned
 *    trajectories take neither step s nor any later step.
 *  - Noise: standard normals from Philox4x32-10 (Salmon et al., SC'11) with
 *    key = (seed low, seed high) and counter = (element / 4, step,
 *    trajectory id, stream id 0); the trajectory id is
 *    (group_offset + g) * N0 + original slot and survives compaction.  The four
 *    output words r0..r3 give elements 4q..4q+3 by Box-Muller on 24-bit
 *    uniforms: u1 = ((r0 >> 8) + 1) / 2^24, u2 = (r1 >> 8) / 2^24,
 *    xi = sqrt(-2 ln u1) * (cos, sin)(2 pi u2); likewise (r2, r3).
 */
#ifndef PROGRPO_H
#define PROGRPO_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define PG_OK          0
#define PG_EINVAL     (-1)  /* bad argument, shape, alignment or null pointer        */
#define PG_ESTATE     (-2)  /* call out of sequence for the handle's schedule          */
#define PG_ECUDA      (-3)  /* a CUDA runtime call failed; see pg_last_cuda_error()    */
#define PG_ENONFINITE (-4)  /* reported by pg_rollout_status(): non-finite scores seen */
#define PG_ETIMEOUT   (-5)  /* reported by pg_rollout_status(): a bounded device wait expired */
#define PG_ENOMEM     (-6)  /* host or device allocation for the handle failed         */
#define PG_EINDEX     (-8)  /* reported by pg_rollout_status(): a gather index was out of range */
#define PG_ECAPACITY  (-7)  /* request larger than a fixed built-in buffer (pg_score_static) */
#define PG_EDEVICE    (-9)  /* the handle was created on another device than the current one  */

#define PG_VEL_F32  0
#define PG_VEL_BF16 1

#define PG_MAX_GROUP 1024   /* largest N0 (trajectories per group) the selection kernels take */
#define PG_MAX_STAGES 32    /* most pruning checkpoints pg_survivor_rows can trace back through */

typedef struct pg_rollout pg_rollout; /* opaque */

/* Schedule of one rollout batch (Section 5.2, "Expand and Prune"). */
typedef struct {
  int32_t n_groups;        /* G  prompt groups handled by this handle                         */
  int32_t n_expand;        /* N0 = G_max trajectories per group at step 0, 1..PG_MAX_GROUP     */
  int32_t elems;           /* d  elements per latent (C*H*W), a positive multiple of 4         */
  int32_t n_steps;         /* T  SDE steps                                                     */
  int32_t n_stages;        /* I  pruning checkpoints (may be 0)                                */
  const int32_t *stage_step; /* [I] strictly increasing, 0 <= step < T                         */
  const int32_t *stage_keep; /* [I] survivors per group, non-increasing, 1 <= keep <= previous  */
  uint64_t seed;           /* Philox key                                                       */
  int32_t group_offset;    /* index of this handle's first group in the whole job (multi-GPU
                              sharding by groups); enters the trajectory id only             */
  int32_t vel_dtype;       /* PG_VEL_F32 or PG_VEL_BF16: element type of every `vel` tensor    */
  int32_t logp_mean;       /* 0: log-density summed over elements; 1: divided by d             */
  float   adv_eps;         /* epsilon of the advantage denominator, >= 0                       */
} pg_config;

/* x' = c_x * x + c_v * v + noise_std * xi.  For drift b = v: c_x = 1, c_v = dt,
 * noise_std = sigma_t * sqrt(dt).  Other backbones (the score-corrected drifts
 * of Eq. "backbone_drifts_method") are affine in (x, prediction) as well and
 * use other coefficients.  Evaluated in fp32 on the device. */
typedef struct { double c_x, c_v, noise_std; } pg_step_coef;

/* x_hat = p_x * x + p_v * v  (Eq. "ode_lookahead_method"; rectified flow:
 * p_x = 1, p_v = remaining time). */
typedef struct { double p_x, p_v; } pg_preview_coef;

/*
 * Creates a handle for one batch (Section 5.1 "Initialization"; Section 5.2).
 * Allocates the handle's device scratch on the current device.  Errors:
 * PG_EINVAL for an inconsistent schedule, PG_ENOMEM / PG_ECUDA.
 */
int pg_rollout_init(const pg_config *cfg, pg_rollout **out);

/* Frees the handle and its scratch.  The caller must have synchronised the
 * stream the handle was used on.  NULL is accepted. */
int pg_rollout_destroy(pg_rollout *h);

/* Rewinds the handle to step 0 / stage 0 with all N0 trajectories active
 * (enqueues the reset of the trajectory-id map on `stream`). */
int pg_rollout_reset(pg_rollout *h, void *stream);

/*
 * Resume from a checkpoint.  The state of a rollout is (latents, next step, stages done,
 * trajectory ids of the active rows, seed); noise is a pure function of (seed, trajectory id,
 * step, element), so a handle restored to that state continues exactly as the interrupted run
 * would have.  traj_ids: device [G * K] int32 with K the survivor count after `stages_done`
 * stages (as returned by pg_rollout_traj_ids at checkpoint time).  The cursor must be reachable:
 * all stages scheduled before next_step done, none scheduled after it (else PG_ESTATE).
 */
int pg_rollout_restore(pg_rollout *h, int32_t next_step, int32_t stages_done, const int32_t *traj_ids,
                       void *stream);

/*
 * Synchronises the device and reports the host-side cursor (trajectories
 * active in total, next step index) and the device status word (bit 0:
 * non-finite score seen by pg_prune_ovf, bit 1: a bounded wait expired, bit 2:
 * a src_rows / keep_idx entry given to pg_step / pg_compact was out of range -
 * such an entry is never dereferenced: pg_step computes that row from row 0,
 * pg_compact leaves it unwritten).  Any out pointer may be NULL.  Returns
 * PG_EINDEX / PG_ETIMEOUT / PG_ENONFINITE if the corresponding bit is set (in
 * that order of precedence), else PG_OK.
 */
int pg_rollout_status(pg_rollout *h, int32_t *n_active, int32_t *next_step, int32_t *device_status);

/*
 * SDE step with fused Gaussian policy log-probability (Eq. "euler_method"; the
 * policy pi_theta of Section 5.1 is the Gaussian N(m, noise_std^2 I) that the
 * step induces).  For each active row i (src = src_rows ? src_rows[i] : i):
 *     m      = c_x * x_in[src] + c_v * vel[src]
 *     x_out[i] = m + noise_std * xi(trajectory id of row i, step)
 *     logp_out[i] = -1/2 * sum_e xi_e^2 - d/2 * ln(2 pi noise_std^2)   (/ d if logp_mean)
 * x_in  [rows_in, d] fp32, vel [rows_in, d] fp32 or bf16 (cfg.vel_dtype);
 * src_rows [n_active] int32 or NULL: gather used on the step that follows a
 * prune, so that survivors need not be moved first (pass pg_prune_ovf's
 * src_rows output; x_out must then not alias x_in).  Without src_rows, x_out
 * may equal x_in.  x_out [n_active, d] fp32; logp_out [n_active] fp32.
 * noise_std == 0 gives the deterministic update and logp_out = 0.
 * `step` must be the handle's next step, and a stage scheduled at `step` must
 * already have been pruned (else PG_ESTATE).  Advances the step cursor.
 */
int pg_step(pg_rollout *h, int32_t step, const pg_step_coef *coef, const float *x_in,
            const void *vel, const int32_t *src_rows, float *x_out, float *logp_out, void *stream);

/*
 * pg_step that also returns the mean of every updated latent: reward_out[i] = mean_e(x_out[i][e]),
 * [n_active] fp32 - the stand-in for the final reward R(x_T, c) of Eq. "advK" when `step` is the last
 * step (the value pg_score(p_x = 1, p_v = 0) would compute from x_out, up to the order of the fp32
 * additions), reduced from the registers that hold x' so that the final latents are not read again.
 * Everything else as pg_step; valid at any step.
 */
int pg_step_reward(pg_rollout *h, int32_t step, const pg_step_coef *coef, const float *x_in,
                   const void *vel, const int32_t *src_rows, float *x_out, float *logp_out,
                   float *reward_out, void *stream);

/*
 * Latent score at a pruning checkpoint (Eq. "ode_lookahead_method", Eq.
 * "proxy_reward_method").  The preview x_hat = p_x * x + p_v * vel is reduced
 * to the stand-in proxy reward r = mean_e(x_hat_e) for each of the n_active
 * rows: scores_out [n_active] fp32.  preview_out (nullable) [n_active, d] fp32
 * receives x_hat for an external decoder / reward model.  With p_v == 0 `vel`
 * is not read and may be NULL (used for the final reward stand-in).  Does not
 * move any cursor; may be called at any time.
 */
int pg_score(pg_rollout *h, const pg_preview_coef *coef, const float *x, const void *vel,
             float *scores_out, float *preview_out, void *stream);

/*
 * Latent score and preview emission in one pass (Eq. "ode_lookahead_method" feeding Eq.
 * "proxy_reward_method": the preview is what the VAE decoder and reward model outside this
 * library consume, the score is the stand-in proxy reward).  Same as pg_score, but the preview
 * is written in the type the consumer wants: preview_dtype PG_VEL_F32 (fp32) or PG_VEL_BF16 (bf16,
 * rounded to nearest even from the fp32 preview), [n_active, d], 16-byte aligned; with bf16
 * the pass moves 8 bytes per element (6 read, 2 written) instead of a 6-byte scoring pass plus an
 * 8-byte pg_preview pass.  scores_out is reduced from the fp32 preview in either case, so it is
 * bit-identical to pg_score's.  preview_out may be NULL (preview_dtype is then ignored).
 */
int pg_score_preview(pg_rollout *h, const pg_preview_coef *coef, const float *x, const void *vel,
                     float *scores_out, void *preview_out, int32_t preview_dtype, void *stream);

/*
 * Preview emission only (Eq. "ode_lookahead_method"): out[i] = p_x * x[i] + p_v * vel[i] for the
 * n_active rows, written as fp32 (out_dtype PG_VEL_F32) or bf16 rounded to nearest even
 * (PG_VEL_BF16), same [n_active, d] layout as the latents, for the VAE decoder and reward model
 * of Eq. "proxy_reward_method" that run outside this library.  No reduction, no cursor change.
 */
int pg_preview(pg_rollout *h, const pg_preview_coef *coef, const float *x, const void *vel, void *out,
               int32_t out_dtype, void *stream);

/*
 * Optimal Variance Filtering for stage `stage` (Eq. "ovf"; Section 5.1): in
 * every group keeps the k = stage_keep[stage] of the K_i active trajectories
 * whose scores have maximal population variance.  The maximiser is found
 * exactly as the best of the k+1 candidates "j lowest and k-j highest" in the
 * total order (score, slot); -0 == +0; NaN orders above +inf; non-finite
 * values enter the variance clamped to +-FLT_MAX and set status bit 0.  Among
 * equal candidates the largest j wins (all-equal scores keep slots 0..k-1).
 * scores [G*K_i] fp32; keep_idx [G*k] int32: kept slots within the group,
 * ascending; src_rows (nullable) [G*k] int32: g*K_i + keep_idx, for pg_step /
 * external gathers; sel_var (nullable) [G] fp32: the selected variance.
 * `stage` must be the next unpruned stage and its step the next step (else
 * PG_ESTATE).  Advances the stage cursor, makes n_active = G*k and compacts the
 * handle's trajectory-id map in stream order.
 */
int pg_prune_ovf(pg_rollout *h, int32_t stage, const float *scores, int32_t *keep_idx,
                 int32_t *src_rows, float *sel_var, void *stream);

/*
 * Uniform-subsampling baseline (Section 4.1, Fig. 1b: k of the G candidates drawn uniformly at random):
 * same contract and cursor effects as pg_prune_ovf, but the k survivors of each group are a
 * uniformly random subset, independent of any score.  Reproducible: slot i of group g draws the
 * first Philox4x32-10 word of counter (i, stage, group_offset + g, stream id 4) under the
 * handle's seed, and the k slots with the smallest (word, slot) are kept, in ascending slot order.
 */
int pg_prune_uniform(pg_rollout *h, int32_t stage, int32_t *keep_idx, int32_t *src_rows, void *stream);

/*
 * Reward-clustering diagnostics (Section 4.1): for each of n_groups groups of n scores the mean
 * mu_G, the population standard deviation sigma_G and the fraction of the group inside the
 * clustered region C_delta = { i : |R_i - mu_G| <= delta * sigma_G } (Eq. "near-mean").
 * scores [n_groups * n] fp32; mean, std, clustered_frac (each nullable) [n_groups] fp32.
 * Stateless; fp64 statistics.
 */
int pg_group_stats(int32_t n_groups, int32_t n, const float *scores, float delta, float *mean,
                   float *std, float *clustered_frac, void *stream);

/*
 * Survivor compaction of a caller-side row array after the most recent
 * pg_prune_ovf (Section 5.1: a pruned trajectory is never stepped again, so
 * only survivors are carried on): dst row g*k + p = src row g*K_prev + keep_idx[g*k + p]; order and
 * count are preserved.  row_bytes > 0; rows need only be byte-aligned, 16-byte
 * aligned rows are moved with 128-bit accesses.  dst must not overlap src.
 */
int pg_compact(pg_rollout *h, const int32_t *keep_idx, const void *src, void *dst,
               size_t row_bytes, void *stream);

/*
 * Group-relative advantages over the survivors (Eq. "advantage", Eq. "advK"):
 * mu = mean, sigma = population standard deviation of the K = n_active / G
 * rewards of a group, adv = (R - mu) / (sigma + adv_eps).  rewards, adv
 * [G*K] fp32; mean, std (nullable) [G] fp32.
 */
int pg_advantages(pg_rollout *h, const float *rewards, float *adv, float *mean, float *std,
                  void *stream);

/*
 * Policy update on the survivors, forward part for one step (Eq. "ratio_method": pi_theta is
 * the Gaussian transition density of the update of Eq. "euler_method"; KL term of Eq.
 * "pro_grpo_method").
 * For each of the n_active rows, with m = c_x x + c_v vel and s = noise_std > 0:
 *     logp_out[i] = -1/2 sum_e ((x_next_e - m_e)/s)^2 - d/2 ln(2 pi s^2)        (/ d if logp_mean)
 *     kl_out[i]   = KL(N(m, s^2 I) || N(m_ref, s^2 I)) = c_v^2 sum_e (vel_e - vel_ref_e)^2 / (2 s^2)
 *                                                                               (/ d if logp_mean)
 * x, x_next [n_active, d] fp32: stored latents before / after the step; vel, vel_ref
 * [n_active, d] in cfg.vel_dtype: new and reference predictions.  vel_ref and kl_out are
 * both NULL or both given.  Read-only pass; uses the handle's reduction scratch (same stream
 * rule as the other calls).  Does not move any cursor.
 * At the rollout's own prediction this is pg_step's logp_out up to fp32 rounding: pg_step reports
 * the density of the sampled action from the generator's radius terms, this call recomputes it
 * from the stored fp32 x_next, and the two differ by at most 2e-6 * d in sum mode (2e-6 with
 * logp_mean) - 0.5 for a 262144-element latent.  Ratios pi_theta / pi_old that must be exactly 1 at
 * theta_old should take both log-probs from this call, or use logp_mean.
 */
int pg_policy_logprob(pg_rollout *h, const pg_step_coef *coef, const float *x, const float *x_next,
                      const void *vel, const void *vel_ref, float *logp_out, float *kl_out, void *stream);

/*
 * Clipped surrogate objective of Eq. "pro_grpo_method" over n_steps steps and the n_active
 * survivors: r = exp(logp_new - logp_old), surr = min(r A, clip(r, 1-clip_eps, 1+clip_eps) A),
 * objective[0] = mean over (step, trajectory) of (surr - beta * kl).  logp_new, logp_old, kl
 * (nullable), ratio (nullable, out), dlogp (out) are [n_steps, n_active] fp32; adv [n_active].
 * dlogp = d objective / d logp_new: A r / (n_steps n_active) where the unclipped branch is
 * active, else 0.  The matching derivative with respect to kl is the constant
 * -beta / (n_steps n_active).  Evaluated in fp64 from the fp32 inputs; one launch of as many
 * CTAs as the entries need, their partial sums combined in a fixed order (the same bits on every
 * run); uses the handle's scratch, so calls on one handle must be ordered like all others.
 */
int pg_policy_objective(pg_rollout *h, int32_t n_steps, const float *logp_new, const float *logp_old,
                        const float *kl, const float *adv, float clip_eps, float beta, float *ratio,
                        float *dlogp, float *objective, void *stream);

/*
 * Gradient of the objective with respect to the new prediction of one step:
 *     grad_e = dlogp[i] * c_v (x_next_e - m_e) / s^2 + dkl * c_v^2 (vel_e - vel_ref_e) / s^2
 * (both terms / d if logp_mean).  dlogp [n_active] is the row of pg_policy_objective's dlogp for
 * this step, dkl the scalar -beta / (n_steps n_active) (ignored when vel_ref is NULL).
 * grad_vel [n_active, d] in cfg.vel_dtype (bf16 rounded to nearest even).
 */
int pg_policy_backward(pg_rollout *h, const pg_step_coef *coef, const float *x, const float *x_next,
                       const void *vel, const void *vel_ref, const float *dlogp, double dkl,
                       void *grad_vel, void *stream);

/*
 * Stateless OVF over many groups in one launch: selection as pg_prune_ovf for
 * n_groups groups of n scores, keeping k; optionally the kept scores and their
 * group-relative advantages (Eq. "advK" applied to the kept scores) in the
 * same kernel.  keep_idx [G*k] int32; kept_scores, adv (nullable) [G*k] fp32;
 * status (nullable) device int32, bit 0 is OR-ed in when a non-finite score is
 * seen.  1 <= k <= n <= PG_MAX_GROUP.
 */
int pg_ovf_select_batched(int32_t n_groups, int32_t n, int32_t k, const float *scores,
                          int32_t *keep_idx, float *kept_scores, float *adv, float adv_eps,
                          int32_t *status, void *stream);

/*
 * Whole rollout from HOST buffers (Section 5.1 + 5.2 end to end): copies x0
 * and, step by step, the predictions to the device (copies overlap compute on
 * a second stream), runs score / OVF / step for every step with the preview
 * mean as score (or host-supplied scores), then the final reward stand-in
 * (mean of x_T, or host-supplied rewards) and the advantages, and copies the
 * results back.  Synchronises before returning.
 *   x0        host [G*N0, d] fp32, or NULL: the initial latents x_0 ~ N(0, I) of Section 5.1 are
 *             then drawn on the device by the library's generator (the rows pg_normal_rows
 *             gives for step 0, noise stream 1 and the global trajectory ids), so no latent
 *             crosses the bus on the way in
 *   vel_steps host array of T pointers; vel_steps[s] is [rows_s, d] in
 *             cfg.vel_dtype with rows_s = rows alive when step s is predicted
 *             (G*K before any prune scheduled at s)
 *   step_coef [T], preview_coef [I] host arrays
 *   stage_scores host array of I pointers to fp32 [rows] or NULL (preview mean)
 *   final_rewards host fp32 [G*K] or NULL (mean of x_T)
 *   outputs (host, any may be NULL): x_final [G*K, d], logp [T][...] packed
 *   step after step (sum over s of rows taking step s), keep_idx packed stage
 *   after stage, adv [G*K], traj_id [G*K].
 *   workspace: device memory of at least pg_rollout_host_workspace_bytes(cfg).
 * Host buffers should be pinned for full copy bandwidth.
 */
size_t pg_rollout_host_workspace_bytes(const pg_config *cfg);
int pg_rollout_host(const pg_config *cfg, const pg_step_coef *step_coef,
                    const pg_preview_coef *preview_coef, const float *x0,
                    const void *const *vel_steps, const float *const *stage_scores,
                    const float *final_rewards, float *x_final, float *logp, int32_t *keep_idx,
                    float *adv, int32_t *traj_id, void *workspace, size_t workspace_bytes);

/*
 * The same whole rollout from HOST buffers on an existing handle (Section 5.1 + 5.2 end to end):
 * pg_rollout_host creates and destroys a handle - six device allocations and a device
 * synchronisation - on every call, which dominates the call for small latents; a caller that
 * rolls out the same schedule repeatedly creates the handle once and calls this instead.  The
 * handle is rewound first; its two streams and four events are created on the first call and
 * released by pg_rollout_destroy, so later calls allocate nothing.  Arguments, layout of the
 * outputs and the workspace are those of pg_rollout_host (schedule = the handle's); synchronises
 * before returning.  The work runs on the handle's own streams: the handle must be idle when
 * the call is made (nothing enqueued on it by the caller still in flight).
 */
int pg_rollout_host_on(pg_rollout *h, const pg_step_coef *step_coef,
                       const pg_preview_coef *preview_coef, const float *x0,
                       const void *const *vel_steps, const float *const *stage_scores,
                       const float *final_rewards, float *x_final, float *logp, int32_t *keep_idx,
                       float *adv, int32_t *traj_id, void *workspace, size_t workspace_bytes);

/*
 * Latent score without any allocation (no counterpart in the paper: this is a packaging
 * variant of pg_score for restricted callers; the arithmetic is that of pg_score).
 *
 * For callers that cannot allocate device memory when they need a score: plug-ins running
 * inside another framework's memory pool, services whose device footprint is fixed at
 * start-up, code in a latency-critical section where cudaMalloc (which may synchronise the
 * device) is unwelcome.  pg_score needs a handle and pg_rollout_init allocates; this call
 * needs neither.  Its reduction scratch is a fixed array inside the library image
 * (about 300 KB, resident on every GPU that loads the library until the process exits).
 *
 *   scores_out[i] = mean_e(p_x * x[i][e] + p_v * vel[i][e]),  i < n_rows
 *   x [n_rows, elems] fp32, vel [n_rows, elems] fp32 or bf16 per vel_dtype (not read and may
 *   be NULL when p_v == 0), scores_out [n_rows] fp32: caller-owned device memory, x and vel
 *   16-byte aligned.  elems a positive multiple of 4.
 *
 * Limits: n_rows <= PG_STATIC_MAX_ROWS and n_rows * ceil(elems / 32768) <=
 * PG_STATIC_MAX_PARTIALS; beyond either the call returns PG_ECAPACITY and does nothing
 * (split the rows over several calls).  Calls no cudaMalloc / cudaFree.  The first call on
 * each device looks up the device address of the built-in array; make that first call
 * outside any stream capture.  All calls on a device share the array and it keeps the last
 * call's contents (the call clears the counters it needs in stream order), so two calls
 * whose kernels can overlap on the GPU (different streams, no ordering) race: keep calls
 * on one stream or order them with events.
 */
#define PG_STATIC_MAX_ROWS     8192
#define PG_STATIC_MAX_PARTIALS 65536
int pg_score_static(int32_t n_rows, int32_t elems, int32_t vel_dtype, const pg_preview_coef *coef,
                    const float *x, const void *vel, float *scores_out, void *stream);

/*
 * Whole rollout from DEVICE buffers on an existing handle (Section 5.1 + 5.2 end to end): resets
 * the handle, then enqueues score / OVF / step for every step and the final reward stand-in and
 * advantages, all on `stream`, without synchronising and without allocating - the sequence of
 * launches is fixed by the schedule, so a caller may capture the call in a CUDA graph and replay
 * it (the usual remedy when the latents are small and the rollout is launch-bound).
 *   x0 device [G*N0, d] fp32 (only read); vel_steps HOST array of T device pointers, vel_steps[s]
 *   being [rows_s, d] in cfg.vel_dtype (rows_s as for pg_rollout_host); stage_scores NULL or a
 *   HOST array of I device pointers (NULL entry = preview mean); final_rewards device or NULL.
 *   workspace: device memory of at least pg_rollout_run_workspace_bytes(cfg) bytes, 16-byte
 *   aligned; results live inside it and are described by *out (device pointers; logp packed step
 *   after step, keep_idx stage after stage).
 */
typedef struct {
  const float *x_final;      /* [n_final, d]          */
  const float *logp;         /* [n_logp]              */
  const int32_t *keep_idx;   /* [n_keep]              */
  const float *adv;          /* [n_final]             */
  const float *rewards;      /* [n_final]             */
  const int32_t *traj_id;    /* [n_final]             */
  int32_t n_final;
  int64_t n_logp, n_keep;
} pg_rollout_outputs;
size_t pg_rollout_run_workspace_bytes(const pg_config *cfg);
int pg_rollout_run(pg_rollout *h, const pg_step_coef *step_coef, const pg_preview_coef *preview_coef,
                   const float *x0, const void *const *vel_steps, const float *const *stage_scores,
                   const float *final_rewards, void *workspace, size_t workspace_bytes,
                   pg_rollout_outputs *out, void *stream);

/* Copies the handle's current trajectory-id map ([n_active] int32, device
 * memory) to `dst` (device) in stream order. */
int pg_rollout_traj_ids(pg_rollout *h, int32_t *dst, void *stream);

/*
 * The survivors' history (Section 5.1, "GRPO with the pruned trajectory set"): the objective of
 * Eq. "pro_grpo_method" runs over the final survivors only, but over all T steps, so a trainer
 * needs the survivors' log-probs and latents also from the steps before a prune, when they sat
 * among rows that were dropped later.
 *
 * pg_survivor_rows: rows_out [T, G*K] int32 (device); rows_out[t][g*K + j] is the row, among the
 *   G*K_t rows that took step t (group-major), of the j-th final survivor of group g.  Depends
 *   only on the handle's schedule and on keep_idx_packed: the kept-slot lists of all stages as
 *   pg_prune_ovf wrote them, packed stage after stage ([G*k_1], [G*k_2], ...; device; may be NULL
 *   without stages), not on the cursor.  A kept slot outside its group is not followed: status
 *   bit 2 / PG_EINDEX.  More than PG_MAX_STAGES stages: PG_ECAPACITY.
 * pg_survivor_logp: logp_out [T, G*K] fp32 = the survivors' entries of the per-step log-prob
 *   arrays packed step after step (logp_packed, sum over t of G*K_t entries, as pg_rollout_run
 *   and pg_rollout_host lay them out), picked through `rows` from pg_survivor_rows.
 * pg_gather_rows: dst row j = src row rows[j] for j < n_out (rows of row_bytes bytes, src has
 *   n_in rows, no overlap): with rows_out[t-1] (or the survivors' original rows for t = 0) this
 *   collects the survivors' x_t from a stored step.  Out-of-range entries are skipped and
 *   reported as PG_EINDEX by pg_rollout_status.
 */
int pg_survivor_rows(pg_rollout *h, const int32_t *keep_idx_packed, int32_t *rows_out, void *stream);
int pg_survivor_logp(pg_rollout *h, const int32_t *rows, const float *logp_packed, float *logp_out,
                     void *stream);
int pg_gather_rows(pg_rollout *h, const int32_t *rows, int32_t n_out, int32_t n_in, const void *src,
                   void *dst, size_t row_bytes, void *stream);

/*
 * Diagnostic (the paper has no counterpart): exercises the library's bounded device-side wait.
 * The only wait inside the kernels is the selection kernel's wait for its score rows to land in
 * shared memory; it gives up after a fixed number of attempts, sets status bit 1 and lets the
 * kernel return, so that a lost copy shows up as PG_ETIMEOUT from pg_rollout_status instead of a
 * hung GPU.  This call launches one warp that waits the same way on a barrier nothing completes:
 * the wait runs out (a fraction of a second at most), bit 1 of the handle's status word is set,
 * and the next pg_rollout_status returns PG_ETIMEOUT.  pg_rollout_reset clears the word.
 */
int pg_selftest_bounded_wait(pg_rollout *h, void *stream);

/* Raw Philox4x32-10 blocks for n (counter, key) pairs: ctr [n,4], key [n,2],
 * out [n,4] uint32 device arrays.  Exposes the library's generator so that it
 * can be compared bit for bit with another implementation. */
int pg_philox_raw(int64_t n, const uint32_t *ctr, const uint32_t *key, uint32_t *out, void *stream);

/* Standard normals exactly as pg_step draws them: out [n_rows, d] fp32 for
 * trajectory ids traj_id [n_rows] (device) at `step`, stream id `stream_id`. */
int pg_normal_rows(uint64_t seed, int32_t step, int32_t stream_id, int32_t n_rows, int32_t d,
                   const int32_t *traj_id, float *out, void *stream);

const char *pg_strerror(int code);
int pg_last_cuda_error(void);
/* Number of kernels the library has launched so far from the calling process. */
uint64_t pg_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* PROGRPO_H */
