/*
 * CPU oracle for the Expand-and-Prune rollout arithmetic of Pro-GRPO.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, double-precision
 * statement of what the GPU library must compute.  It is compiled by gcc into
 * its own shared object, shares no source, header, table or helper with the
 * CUDA code, and is called only from the tests, the smoke check and the CPU
 * baseline leg of the benchmark.  Nothing here is tuned; OpenMP is used only
 * to spread independent trajectories / groups over host cores.
 *
 * Every function names the passage of the paper it follows.  Floating point
 * is IEEE double throughout; fp32 / bf16 occur only where a value enters or
 * leaves (latents are stored as fp32 between steps because the rollout state
 * is fp32).  Compile with -ffp-contract=off so that no fused multiply-add is
 * formed behind the stated order of operations.
 *
 * Parity pins (tests/test_oracle_*.py): Philox known answers, normal-sample
 * statistics, Gaussian log-density against scipy, moment recursions of the
 * Euler-Maruyama step, exhaustive subset search for OVF, numpy statistics
 * for the advantages; for the policy update scipy densities, a numerically
 * integrated KL, hand-worked clipping cases and finite differences.  No
 * function in this file is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <float.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define OG_OK 0
#define OG_EINVAL (-1)

/* ------------------------------------------------------------------ */
/* Counter-based noise                                                 */
/* ------------------------------------------------------------------ */

/*
 * Philox4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw: "Parallel random
 * numbers: as easy as 1, 2, 3", SC'11, Section 3.3 / Table 2 constants).
 * One round: the two 32x32->64 products of (M0, ctr[0]) and (M1, ctr[2])
 * are split into high and low words and recombined with the key; the key is
 * bumped by the Weyl constants between rounds.
 */
void og_philox4x32_10(const uint32_t ctr_in[4], const uint32_t key_in[2], uint32_t out[4])
{
    const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
    const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
    uint32_t c0 = ctr_in[0], c1 = ctr_in[1], c2 = ctr_in[2], c3 = ctr_in[3];
    uint32_t k0 = key_in[0], k1 = key_in[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) { k0 += W0; k1 += W1; }
        uint64_t p0 = (uint64_t)M0 * (uint64_t)c0;
        uint64_t p1 = (uint64_t)M1 * (uint64_t)c2;
        uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/*
 * Standard normals for the four elements 4q .. 4q+3 of one trajectory at one
 * step.  The noise of the Euler-Maruyama update (Eq. "euler_method":
 * xi ~ N(0, I)) is keyed by (seed, trajectory, step, element):
 *   key     = (seed low word, seed high word)
 *   counter = (q, step, trajectory, stream)
 * Two 24-bit uniforms per pair, Box-Muller:
 *   u1 = ((r >> 8) + 1) / 2^24 in (0, 1],  u2 = (r' >> 8) / 2^24 in [0, 1)
 *   xi_a = sqrt(-2 ln u1) cos(2 pi u2),  xi_b = sqrt(-2 ln u1) sin(2 pi u2)
 */
void og_normal4(uint64_t seed, uint32_t q, uint32_t step, uint32_t trajectory,
                uint32_t stream, double xi[4])
{
    uint32_t ctr[4] = { q, step, trajectory, stream };
    uint32_t key[2] = { (uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32) };
    uint32_t r[4];
    og_philox4x32_10(ctr, key, r);
    const double two_pi = 6.283185307179586476925286766559;
    const double scale = 1.0 / 16777216.0; /* 2^-24 */
    for (int p = 0; p < 2; ++p) {
        double u1 = ((double)(r[2 * p] >> 8) + 1.0) * scale;
        double u2 = (double)(r[2 * p + 1] >> 8) * scale;
        double radius = sqrt(-2.0 * log(u1));
        double angle = two_pi * u2;
        xi[2 * p] = radius * cos(angle);
        xi[2 * p + 1] = radius * sin(angle);
    }
}

/* Raw generator words for many (counter, key) pairs; used by the bit-exact
 * comparison against the GPU generator. */
void og_philox_batch(int64_t n, const uint32_t *ctr /*[n,4]*/, const uint32_t *key /*[n,2]*/,
                     uint32_t *out /*[n,4]*/)
{
    for (int64_t i = 0; i < n; ++i)
        og_philox4x32_10(ctr + 4 * i, key + 2 * i, out + 4 * i);
}

/* Normals for one whole (trajectory, step): d values, d a multiple of 4. */
int og_normal_row(uint64_t seed, uint32_t step, uint32_t trajectory, uint32_t stream,
                  int64_t d, double *xi_out)
{
    if (d < 0 || (d & 3)) return OG_EINVAL;
    for (int64_t q = 0; q < d / 4; ++q)
        og_normal4(seed, (uint32_t)q, step, trajectory, stream, xi_out + 4 * q);
    return OG_OK;
}

/* ------------------------------------------------------------------ */
/* Input decoding                                                      */
/* ------------------------------------------------------------------ */

static double bf16_to_double(uint16_t h)
{
    uint32_t bits = (uint32_t)h << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

/* vel_dtype: 0 = fp32, 1 = bf16 (raw 16-bit words). */
static double load_vel(const void *vel, int vel_dtype, int64_t index)
{
    if (vel_dtype == 1) return bf16_to_double(((const uint16_t *)vel)[index]);
    return (double)((const float *)vel)[index];
}

/* ------------------------------------------------------------------ */
/* SDE step and Gaussian policy log-probability                        */
/* ------------------------------------------------------------------ */

/*
 * One Euler-Maruyama step of the unified reverse SDE (Eq. "unified_sde_method",
 * Eq. "euler_method") for n active trajectories of d elements:
 *     mean  m  = c_x * x + c_v * v          ( = x + b_theta * dt )
 *     x'       = m + noise_std * xi          ( noise_std = sigma_t * sqrt(dt) )
 * and the log-density of the Gaussian policy that this step induces
 * (Section 5.1, text under Eq. "ratio_method": pi is N(m, noise_std^2 I)):
 *     log pi = -1/2 * sum_e ((x'_e - m_e) / noise_std)^2 - d/2 * ln(2 pi noise_std^2)
 * With logp_mean != 0 the sum is divided by d.
 *
 * Row i of the output reads row src = src_slot ? src_slot[i] : i of x_in and
 * vel (early-terminated trajectories are simply never read again), and draws
 * its noise with trajectory id traj_id[i], so the noise of a trajectory does
 * not depend on where compaction has moved it.
 *
 * noise_std == 0 gives the deterministic update; the density is then
 * degenerate and logp is reported as 0.
 */
int og_step(int64_t n, int64_t d,
            const float *x_in, const void *vel, int vel_dtype,
            const int32_t *src_slot, const int32_t *traj_id,
            uint64_t seed, uint32_t step,
            double c_x, double c_v, double noise_std, int logp_mean,
            float *x_out, double *logp_out)
{
    if (n < 0 || d <= 0 || (d & 3) || !x_in || !vel || !traj_id || !x_out || !logp_out)
        return OG_EINVAL;
    if (!(noise_std >= 0.0)) return OG_EINVAL;
    const double two_pi = 6.283185307179586476925286766559;
    #pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < n; ++i) {
        int64_t src = src_slot ? (int64_t)src_slot[i] : i;
        const float *x_row = x_in + src * d;
        float *o_row = x_out + i * d;
        double sum_sq = 0.0;
        for (int64_t q = 0; q < d / 4; ++q) {
            double xi[4];
            og_normal4(seed, (uint32_t)q, step, (uint32_t)traj_id[i], 0u, xi);
            for (int j = 0; j < 4; ++j) {
                int64_t e = 4 * q + j;
                double x = (double)x_row[e];
                double v = load_vel(vel, vel_dtype, src * d + e);
                double m = c_x * x + c_v * v;
                double x_new = m + noise_std * xi[j];
                if (noise_std > 0.0) {
                    double z = (x_new - m) / noise_std;
                    sum_sq += z * z;
                }
                o_row[e] = (float)x_new;
            }
        }
        double lp = 0.0;
        if (noise_std > 0.0) {
            lp = -0.5 * sum_sq - 0.5 * (double)d * log(two_pi * noise_std * noise_std);
            if (logp_mean) lp /= (double)d;
        }
        logp_out[i] = lp;
    }
    return OG_OK;
}

/*
 * Log-density of an arbitrary transition x -> x_next under the same Gaussian
 * policy (used to pin og_step's reported value against the stored latents).
 */
int og_transition_logp(int64_t n, int64_t d, const float *x_in, const void *vel, int vel_dtype,
                       const double *x_next, double c_x, double c_v, double noise_std,
                       int logp_mean, double *logp_out)
{
    if (n < 0 || d <= 0 || !(noise_std > 0.0)) return OG_EINVAL;
    const double two_pi = 6.283185307179586476925286766559;
    for (int64_t i = 0; i < n; ++i) {
        double sum_sq = 0.0;
        for (int64_t e = 0; e < d; ++e) {
            double m = c_x * (double)x_in[i * d + e] + c_v * load_vel(vel, vel_dtype, i * d + e);
            double z = (x_next[i * d + e] - m) / noise_std;
            sum_sq += z * z;
        }
        double lp = -0.5 * sum_sq - 0.5 * (double)d * log(two_pi * noise_std * noise_std);
        logp_out[i] = logp_mean ? lp / (double)d : lp;
    }
    return OG_OK;
}

/* ------------------------------------------------------------------ */
/* ODE look-ahead preview and latent score                             */
/* ------------------------------------------------------------------ */

/*
 * Single-step deterministic projection of each active latent to the terminal
 * time (Eq. "ode_lookahead_method"):  x_hat = p_x * x + p_v * v, where for a
 * rectified-flow backbone p_x = 1 and p_v = remaining time (Eq.
 * "ode_drift_method": b_ODE = v_theta).  The proxy reward of Eq.
 * "proxy_reward_method" needs a decoder and a reward network; the stand-in
 * used throughout this project is the mean of the preview latent,
 *     r = (1/d) * sum_e x_hat_e .
 * preview_out (nullable) receives x_hat rounded to fp32.
 */
int og_score(int64_t n, int64_t d, const float *x, const void *vel, int vel_dtype,
             double p_x, double p_v, double *score_out, float *preview_out)
{
    if (n < 0 || d <= 0 || !x || !vel || !score_out) return OG_EINVAL;
    #pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < n; ++i) {
        double sum = 0.0;
        for (int64_t e = 0; e < d; ++e) {
            double xh = p_x * (double)x[i * d + e] + p_v * load_vel(vel, vel_dtype, i * d + e);
            sum += xh;
            if (preview_out) preview_out[i * d + e] = (float)xh;
        }
        score_out[i] = sum / (double)d;
    }
    return OG_OK;
}

/* ------------------------------------------------------------------ */
/* Optimal Variance Filtering                                          */
/* ------------------------------------------------------------------ */

/* Population variance (1/k) sum (r - mean)^2 of the listed members. */
static double subset_variance(const double *r, const int *members, int k)
{
    double mean = 0.0;
    for (int i = 0; i < k; ++i) mean += r[members[i]];
    mean /= (double)k;
    double acc = 0.0;
    for (int i = 0; i < k; ++i) {
        double dlt = r[members[i]] - mean;
        acc += dlt * dlt;
    }
    return acc / (double)k;
}

/*
 * OVF by its definition (Eq. "ovf"): among all subsets of size k of the n
 * scores, the one with the largest population variance.  Enumerates every
 * combination in lexicographic order; only for small n (n <= 24 accepted).
 * Returns the maximal variance and the first subset (in lexicographic order)
 * that attains it.
 */
int og_ovf_exhaustive(int n, int k, const float *scores, int32_t *best_subset, double *best_var)
{
    if (n < 1 || n > 24 || k < 1 || k > n || !scores || !best_var) return OG_EINVAL;
    double r[24];
    int comb[24];
    for (int i = 0; i < n; ++i) r[i] = (double)scores[i];
    for (int i = 0; i < k; ++i) comb[i] = i;
    double top = -1.0;
    for (;;) {
        double v = subset_variance(r, comb, k);
        if (v > top) {
            top = v;
            if (best_subset) for (int i = 0; i < k; ++i) best_subset[i] = comb[i];
        }
        int pos = k - 1;
        while (pos >= 0 && comb[pos] == n - k + pos) --pos;
        if (pos < 0) break;
        ++comb[pos];
        for (int i = pos + 1; i < k; ++i) comb[i] = comb[i - 1] + 1;
    }
    *best_var = top;
    return OG_OK;
}

/* Total order used by the selection: by score (fp32 value; -0 equals +0; NaN
 * sorts above +inf), ties by slot index. */
typedef struct { float score; int32_t slot; } og_entry;

static int entry_less(const og_entry *a, const og_entry *b)
{
    int a_nan = isnan(a->score), b_nan = isnan(b->score);
    if (a_nan || b_nan) {
        if (a_nan != b_nan) return b_nan;     /* the non-NaN one is lower */
        return a->slot < b->slot;
    }
    if (a->score < b->score) return 1;
    if (a->score > b->score) return 0;
    return a->slot < b->slot;
}

/* Value that enters the variance arithmetic: the score itself, with
 * non-finite values replaced by the nearest finite fp32 (NaN -> +FLT_MAX). */
static double arithmetic_value(float s)
{
    if (isnan(s)) return (double)FLT_MAX;
    if (s > FLT_MAX) return (double)FLT_MAX;
    if (s < -FLT_MAX) return -(double)FLT_MAX;
    return (double)s;
}

/*
 * OVF for any group size (Eq. "ovf", and its in-process form in Section 5.1).
 * The variance of a set is a convex quadratic in each member, so a maximiser
 * always has the shape "the j lowest and the k-j highest scores" (the subset
 * sits at both ends of the score range, as Fig. 1c illustrates).  Steps:
 *   1. order the slots by (score, slot);
 *   2. centre on the score at order position n/2 (keeps the sums small);
 *   3. running sums of c and c*c from the low end (L1, L2) and from the high
 *      end (H1, H2), each accumulated serially one element at a time;
 *   4. for j = 0..k:  S = L1[j] + H1[k-j],  Q = L2[j] + H2[k-j],
 *      M_j = k*Q - S*S   ( = k^2 * variance of that candidate );
 *   5. j* = the largest j whose M_j is maximal;
 *   6. keep the first j* and the last k-j* of the order, report kept slots in
 *      ascending slot order, variance M_j* / k^2.
 */
int og_ovf_select(int n, int k, const float *scores, int32_t *keep_idx, double *sel_var,
                  int32_t *low_count)
{
    if (n < 1 || k < 1 || k > n || !scores || !keep_idx) return OG_EINVAL;
    og_entry *order = (og_entry *)malloc((size_t)n * sizeof(og_entry));
    double *L1 = (double *)malloc((size_t)(k + 1) * 4 * sizeof(double));
    unsigned char *keep = (unsigned char *)calloc((size_t)n, 1);
    if (!order || !L1 || !keep) { free(order); free(L1); free(keep); return OG_EINVAL; }
    double *L2 = L1 + (k + 1), *H1 = L2 + (k + 1), *H2 = H1 + (k + 1);

    for (int i = 0; i < n; ++i) { order[i].score = scores[i]; order[i].slot = i; }
    /* insertion sort: plain, stable with respect to the explicit total order */
    for (int i = 1; i < n; ++i) {
        og_entry cur = order[i];
        int p = i - 1;
        while (p >= 0 && entry_less(&cur, &order[p])) { order[p + 1] = order[p]; --p; }
        order[p + 1] = cur;
    }
    double pivot = arithmetic_value(order[n / 2].score);

    L1[0] = L2[0] = H1[0] = H2[0] = 0.0;
    for (int j = 1; j <= k; ++j) {
        double c = arithmetic_value(order[j - 1].score) - pivot;
        double cc = c * c;
        L1[j] = L1[j - 1] + c;
        L2[j] = L2[j - 1] + cc;
    }
    for (int m = 1; m <= k; ++m) {
        double c = arithmetic_value(order[n - m].score) - pivot;
        double cc = c * c;
        H1[m] = H1[m - 1] + c;
        H2[m] = H2[m - 1] + cc;
    }
    int best_j = 0;
    double best_m = 0.0;
    for (int j = 0; j <= k; ++j) {
        double S = L1[j] + H1[k - j];
        double Q = L2[j] + H2[k - j];
        double kq = (double)k * Q;
        double ss = S * S;
        double M = kq - ss;
        if (j == 0 || M >= best_m) { best_m = M; best_j = j; }
    }
    for (int j = 0; j < best_j; ++j) keep[order[j].slot] = 1;
    for (int m = 1; m <= k - best_j; ++m) keep[order[n - m].slot] = 1;
    int w = 0;
    for (int i = 0; i < n; ++i) if (keep[i]) keep_idx[w++] = i;
    if (sel_var) *sel_var = best_m / ((double)k * (double)k);
    if (low_count) *low_count = best_j;
    free(order); free(L1); free(keep);
    return (w == k) ? OG_OK : OG_EINVAL;
}

/* og_ovf_select over G independent groups of n scores each. */
int og_ovf_select_groups(int n_groups, int n, int k, const float *scores,
                         int32_t *keep_idx /*[G,k]*/, double *sel_var /*nullable [G]*/)
{
    if (n_groups < 0) return OG_EINVAL;
    int status = OG_OK;
    #pragma omp parallel for schedule(static)
    for (int g = 0; g < n_groups; ++g) {
        int rc = og_ovf_select(n, k, scores + (size_t)g * n, keep_idx + (size_t)g * k,
                               sel_var ? sel_var + g : NULL, NULL);
        if (rc != OG_OK) {
            #pragma omp critical
            status = rc;
        }
    }
    return status;
}

/* ------------------------------------------------------------------ */
/* Compaction                                                          */
/* ------------------------------------------------------------------ */

/*
 * Early termination (Section 5.1: a pruned trajectory is never stepped
 * again): the survivors of each group become a dense block, in ascending
 * slot order.  Row g*k + p of dst is row g*n_prev + keep_idx[g*k + p] of src.
 */
int og_compact_rows(int n_groups, int n_prev, int k, const int32_t *keep_idx,
                    const void *src, void *dst, size_t row_bytes)
{
    if (n_groups < 0 || n_prev < 1 || k < 1 || k > n_prev || !keep_idx || !src || !dst)
        return OG_EINVAL;
    for (int g = 0; g < n_groups; ++g)
        for (int p = 0; p < k; ++p) {
            int32_t slot = keep_idx[(size_t)g * k + p];
            if (slot < 0 || slot >= n_prev) return OG_EINVAL;
            memcpy((char *)dst + ((size_t)g * k + p) * row_bytes,
                   (const char *)src + ((size_t)g * n_prev + slot) * row_bytes, row_bytes);
        }
    return OG_OK;
}

/* ------------------------------------------------------------------ */
/* Group-relative advantages                                           */
/* ------------------------------------------------------------------ */

/*
 * Eq. "advantage" / Eq. "advK": per group of K rewards,
 *   mu = (1/K) sum R,  sigma = sqrt((1/K) sum (R - mu)^2),  A = (R - mu) / (sigma + eps).
 */
int og_advantages(int n_groups, int K, const float *rewards, double eps,
                  double *adv, double *mean_out, double *std_out)
{
    if (n_groups < 0 || K < 1 || !rewards || !adv) return OG_EINVAL;
    for (int g = 0; g < n_groups; ++g) {
        const float *r = rewards + (size_t)g * K;
        double mu = 0.0;
        for (int i = 0; i < K; ++i) mu += (double)r[i];
        mu /= (double)K;
        double acc = 0.0;
        for (int i = 0; i < K; ++i) {
            double dlt = (double)r[i] - mu;
            acc += dlt * dlt;
        }
        double sigma = sqrt(acc / (double)K);
        for (int i = 0; i < K; ++i)
            adv[(size_t)g * K + i] = ((double)r[i] - mu) / (sigma + eps);
        if (mean_out) mean_out[g] = mu;
        if (std_out) std_out[g] = sigma;
    }
    return OG_OK;
}

int og_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------ */
/* Policy update on the survivors (Section 5.1, Eq. "ratio_method",    */
/* Eq. "pro_grpo_method"; GRPO loss of Section 3.3)                    */
/* ------------------------------------------------------------------ */

/*
 * Log-density of the stored transition x -> x_next under the Gaussian policy
 * that a (new) prediction `vel` induces, and the KL divergence from the policy
 * of a reference prediction `vel_ref`:
 *     m      = c_x x + c_v vel ,   m_ref = c_x x + c_v vel_ref
 *     log pi = -1/2 sum ((x_next - m)/s)^2 - d/2 ln(2 pi s^2)        (/ d if logp_mean)
 *     KL( N(m, s^2 I) || N(m_ref, s^2 I) ) = sum (m - m_ref)^2 / (2 s^2)   (/ d if logp_mean)
 * (two Gaussians with the same covariance: only the mean shift contributes).
 * vel_ref and kl_out may be NULL together.
 */
int og_policy_logprob(int64_t n, int64_t d, const float *x, const float *x_next,
                      const void *vel, const void *vel_ref, int vel_dtype,
                      double c_x, double c_v, double noise_std, int logp_mean,
                      double *logp_out, double *kl_out)
{
    if (n < 0 || d <= 0 || !x || !x_next || !vel || !logp_out || !(noise_std > 0.0)) return OG_EINVAL;
    if ((vel_ref == NULL) != (kl_out == NULL)) return OG_EINVAL;
    const double two_pi = 6.283185307179586476925286766559;
    #pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < n; ++i) {
        double sum_sq = 0.0, sum_kl = 0.0;
        for (int64_t e = 0; e < d; ++e) {
            double xe = (double)x[i * d + e];
            double m = c_x * xe + c_v * load_vel(vel, vel_dtype, i * d + e);
            double z = ((double)x_next[i * d + e] - m) / noise_std;
            sum_sq += z * z;
            if (vel_ref) {
                double m_ref = c_x * xe + c_v * load_vel(vel_ref, vel_dtype, i * d + e);
                double dm = m - m_ref;
                sum_kl += dm * dm;
            }
        }
        double lp = -0.5 * sum_sq - 0.5 * (double)d * log(two_pi * noise_std * noise_std);
        double kl = sum_kl / (2.0 * noise_std * noise_std);
        if (logp_mean) { lp /= (double)d; kl /= (double)d; }
        logp_out[i] = lp;
        if (kl_out) kl_out[i] = kl;
    }
    return OG_OK;
}

/*
 * Clipped surrogate objective over T steps and n trajectories (Eq. "pro_grpo_method"):
 *     r[t,i]   = exp(logp_new[t,i] - logp_old[t,i])                       (Eq. "ratio_method")
 *     surr     = min( r A_i , clip(r, 1-eps, 1+eps) A_i )
 *     J        = mean over (t,i) of ( surr - beta * kl[t,i] )
 * Also the derivative dJ/dlogp_new[t,i]: (1/(nT)) * A_i * r where the unclipped branch is
 * the active one (r A <= clip(r) A, which includes the whole interior of the clip range),
 * else 0.  kl may be NULL (beta term dropped).
 */
int og_policy_objective(int64_t T, int64_t n, const double *logp_new, const double *logp_old,
                        const double *kl, const double *adv, double clip_eps, double beta,
                        double *ratio_out, double *dlogp_out, double *objective_out)
{
    if (T <= 0 || n <= 0 || !logp_new || !logp_old || !adv || !objective_out || !(clip_eps >= 0.0))
        return OG_EINVAL;
    double total = 0.0;
    const double inv = 1.0 / ((double)T * (double)n);
    for (int64_t t = 0; t < T; ++t)
        for (int64_t i = 0; i < n; ++i) {
            int64_t j = t * n + i;
            double r = exp(logp_new[j] - logp_old[j]);
            double lo = 1.0 - clip_eps, hi = 1.0 + clip_eps;
            double rc = r < lo ? lo : (r > hi ? hi : r);
            double a = adv[i];
            double s1 = r * a, s2 = rc * a;
            double surr = s1 < s2 ? s1 : s2;
            total += surr - (kl ? beta * kl[j] : 0.0);
            if (ratio_out) ratio_out[j] = r;
            if (dlogp_out) dlogp_out[j] = (s1 <= s2) ? inv * a * r : 0.0;
        }
    *objective_out = total * inv;
    return OG_OK;
}

/*
 * Gradient of J with respect to the new prediction at one step, given dJ/dlogp of that step
 * (dlogp[i]) and dJ/dkl (a scalar, -beta/(nT)):
 *     dlogp/dvel_e = c_v (x_next_e - m_e) / s^2          (/ d if logp_mean)
 *     dkl/dvel_e   = c_v^2 (vel_e - vel_ref_e) / s^2     (/ d if logp_mean)
 */
int og_policy_backward(int64_t n, int64_t d, const float *x, const float *x_next,
                       const void *vel, const void *vel_ref, int vel_dtype,
                       double c_x, double c_v, double noise_std, int logp_mean,
                       const double *dlogp, double dkl, double *grad_out)
{
    if (n < 0 || d <= 0 || !x || !x_next || !vel || !dlogp || !grad_out || !(noise_std > 0.0))
        return OG_EINVAL;
    const double inv_s2 = 1.0 / (noise_std * noise_std);
    const double scale = logp_mean ? 1.0 / (double)d : 1.0;
    #pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < n; ++i)
        for (int64_t e = 0; e < d; ++e) {
            double v = load_vel(vel, vel_dtype, i * d + e);
            double m = c_x * (double)x[i * d + e] + c_v * v;
            double g = dlogp[i] * c_v * ((double)x_next[i * d + e] - m) * inv_s2;
            if (vel_ref)
                g += dkl * c_v * c_v * (v - load_vel(vel_ref, vel_dtype, i * d + e)) * inv_s2;
            grad_out[i * d + e] = g * scale;
        }
    return OG_OK;
}

/* ------------------------------------------------------------------ */
/* Diagnostics and the uniform-subsampling baseline (Section 4)        */
/* ------------------------------------------------------------------ */

/*
 * Reward-clustering diagnostics per group (Section 4.1): mean mu_G, population standard
 * deviation sigma_G and the fraction of the group inside the clustered region
 *     C_delta = { i : |R_i - mu_G| <= delta * sigma_G }          (Eq. "near-mean").
 */
int og_group_stats(int n_groups, int n, const float *scores, double delta,
                   double *mean_out, double *std_out, double *clustered_out)
{
    if (n_groups < 0 || n < 1 || !scores || !(delta >= 0.0)) return OG_EINVAL;
    for (int g = 0; g < n_groups; ++g) {
        const float *r = scores + (size_t)g * n;
        double mu = 0.0;
        for (int i = 0; i < n; ++i) mu += (double)r[i];
        mu /= (double)n;
        double acc = 0.0;
        for (int i = 0; i < n; ++i) { double dl = (double)r[i] - mu; acc += dl * dl; }
        double sigma = sqrt(acc / (double)n);
        int inside = 0;
        for (int i = 0; i < n; ++i) if (fabs((double)r[i] - mu) <= delta * sigma) ++inside;
        if (mean_out) mean_out[g] = mu;
        if (std_out) std_out[g] = sigma;
        if (clustered_out) clustered_out[g] = (double)inside / (double)n;
    }
    return OG_OK;
}

/*
 * Uniform subsampling of k of n trajectories per group (the baseline of Section 4.1 and
 * Fig. 1b), made reproducible with the counter-based generator: slot i of group `group`
 * draws the word r_i = first output word of Philox4x32-10 with counter
 * (i, stage, group, stream 4) and the seed as key; the k slots with the smallest (r_i, i)
 * are kept and reported in ascending slot order.  Distinct words are equally likely to
 * fall in any order, so every k-subset is equally likely.
 */
int og_select_uniform(int n_groups, int n, int k, uint64_t seed, uint32_t stage,
                      uint32_t group_offset, int32_t *keep_idx)
{
    if (n_groups < 0 || n < 1 || k < 1 || k > n || !keep_idx) return OG_EINVAL;
    uint32_t *word = (uint32_t *)malloc((size_t)n * sizeof(uint32_t));
    if (!word) return OG_EINVAL;
    uint32_t key[2] = { (uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32) };
    for (int g = 0; g < n_groups; ++g) {
        for (int i = 0; i < n; ++i) {
            uint32_t ctr[4] = { (uint32_t)i, stage, group_offset + (uint32_t)g, 4u };
            uint32_t out[4];
            og_philox4x32_10(ctr, key, out);
            word[i] = out[0];
        }
        int w = 0;
        for (int i = 0; i < n; ++i) {
            int smaller = 0;
            for (int j = 0; j < n; ++j)
                if (word[j] < word[i] || (word[j] == word[i] && j < i)) ++smaller;
            if (smaller < k) keep_idx[(size_t)g * k + w++] = i;
        }
        if (w != k) { free(word); return OG_EINVAL; }
    }
    free(word);
    return OG_OK;
}
