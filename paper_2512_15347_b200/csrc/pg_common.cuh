// Shared device helpers and launcher declarations of the Pro-GRPO rollout library (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

#include "../../include/progrpo.h"

namespace pg {

// ---------------------------------------------------------------- host-side bookkeeping
void note_launch();                 // counts kernels launched by the library
int  cuda_fail(cudaError_t e);      // remembers e for pg_last_cuda_error(), returns PG_ECUDA

#define PG_CUDA(call)                                        \
  do {                                                       \
    cudaError_t pg_e_ = (call);                              \
    if (pg_e_ != cudaSuccess) return ::pg::cuda_fail(pg_e_); \
  } while (0)

#define PG_LAUNCH_CHECK()                                    \
  do {                                                       \
    ::pg::note_launch();                                     \
    cudaError_t pg_e_ = cudaGetLastError();                  \
    if (pg_e_ != cudaSuccess) return ::pg::cuda_fail(pg_e_); \
  } while (0)

// ---------------------------------------------------------------- Philox4x32-10
// Round keys k + r * (0x9E3779B9, 0xBB67AE85), r = 0..9, precomputed on the host so that the
// device reads them as immediates from the kernel-parameter bank.
struct PhiloxKeys {
  uint32_t k0[10];
  uint32_t k1[10];
};

inline PhiloxKeys make_philox_keys(uint64_t seed) {
  PhiloxKeys rk;
  uint32_t a = (uint32_t)(seed & 0xFFFFFFFFull), b = (uint32_t)(seed >> 32);
  for (int r = 0; r < 10; ++r) {
    rk.k0[r] = a;
    rk.k1[r] = b;
    a += 0x9E3779B9u;
    b += 0xBB67AE85u;
  }
  return rk;
}

#ifdef __CUDACC__
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                               const PhiloxKeys& rk) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
    const uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
    const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ rk.k0[r];
    const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ rk.k1[r];
    c1 = (uint32_t)p1;
    c3 = (uint32_t)p0;
    c0 = n0;
    c2 = n2;
  }
  return make_uint4(c0, c1, c2, c3);
}

// Box-Muller on two generator words (24-bit uniforms):
//   u1 = ((r0 >> 8) + 1) * 2^-24 in (0, 1],  u2 = (r1 >> 8) * 2^-24 in [0, 1)
//   normals  a = sqrt(-2 ln u1) cos(2 pi u2),  b = sqrt(-2 ln u1) sin(2 pi u2)
// Returned in factored and scaled form: with neg_scale2 = -2 ln 2 * scale^2 the outputs are
// radius = scale * sqrt(-2 ln u1) and (c, s) = (cos, sin)(2 pi u2 - pi), so that scale * a =
// -radius * c and scale * b = -radius * s (half-turn shift: the hardware sine is evaluated on
// [-pi, pi), its most accurate range); the return value is log2(u1) <= 0, i.e. a^2 + b^2 =
// -2 ln 2 * (return value).  Keeping the logarithm in base 2 until the square root saves a
// multiplication per pair: the caller sums the returned values and applies -2 ln 2 once.
// The logarithm uses the hardware log2 except close to u1 = 1, where its absolute error would
// dominate the small radius: there log2(1 - w) is summed as a short series in w = 1 - u1 (w is
// exact in fp32; truncation below 1e-6 relative for w < 2^-6).
constexpr float kTwoLn2 = 1.3862943611198906f;
__device__ __forceinline__ float box_muller(uint32_t r0, uint32_t r1, float neg_scale2, float& radius, float& c,
                                            float& s) {
  const float k1 = (float)(r0 >> 8);
  const float u1 = fmaf(k1, 5.9604644775390625e-8f, 5.9604644775390625e-8f);
  float lg;                                                     // u1 >= 2^-24: never subnormal
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(lg) : "f"(u1));
  const float w = 1.0f - u1;                                     // exact (24-bit grid)
  // log2(1 - w) = -(w + w^2/2 + w^3/3 + ...) / ln 2; the first dropped term is below 1e-6 of the sum
  // for w < 2^-6, i.e. below 1e-7 absolute in the radius, which is then at most 0.18
  float ser = fmaf(w, -0.48089834696298783f, -0.7213475204444817f);
  ser = fmaf(ser, w, -1.4426950408889634f);
  ser *= w;
  lg = (w < 0.015625f) ? ser : lg;
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(radius) : "f"(lg * neg_scale2));
  const float turn = fmaf((float)(r1 >> 8), 5.9604644775390625e-8f, -0.5f);  // u2 - 1/2, exact
  // The cosine is taken as a sine: cos t = sin(pi/2 - |t|), i.e. the sine at 1/4 - |turn| turns
  // (an exact difference on the 24-bit grid, and an argument in [-pi/2, pi/2]).  The hardware
  // sine's error is an odd function of the angle, so over the symmetric angle grid it averages to
  // zero; the hardware cosine's error is even and does not (measured mean +5.8e-8, i.e. -7.2e-8
  // on every cosine normal) - small against the 2e-7 rms error of a draw, but a bias is what the
  // mean of a long latent (the latent score) accumulates over many steps.
  const float angle = 6.283185307179586f * turn;
  const float angle_c = 6.283185307179586f * (0.25f - fabsf(turn));
  asm("sin.approx.ftz.f32 %0, %1;" : "=f"(s) : "f"(angle));
  asm("sin.approx.ftz.f32 %0, %1;" : "=f"(c) : "f"(angle_c));
  return lg;
}

// The two normals themselves.
__device__ __forceinline__ void normal_pair(uint32_t r0, uint32_t r1, float& a, float& b) {
  float radius, c, s;
  box_muller(r0, r1, -kTwoLn2, radius, c, s);
  a = -radius * c;
  b = -radius * s;
}

// Bounded wait on an mbarrier in shared memory (`bar` = shared-space address) for the phase of
// the given parity: up to `limit` try_wait attempts.  Returns true once the phase has completed,
// false when the attempts ran out - the caller then records the timeout and leaves; no wait in
// this library is unbounded.
__device__ __forceinline__ bool mbarrier_wait_bounded(unsigned int bar, unsigned int parity, int limit) {
  unsigned int done = 0;
  for (int it = 0; it < limit && !done; ++it) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
  }
  return done != 0;
}
constexpr int kBulkWaitLimit = 1 << 14;   // try_wait attempts per round before giving up

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}
#endif  // __CUDACC__

// ---------------------------------------------------------------- launch geometry
// Row-streaming kernels (step, score, policy log-prob): a CTA of kRowThreads threads handles one
// chunk of one row and contributes one partial sum, so a row owns `chunks` partial slots.  Chunks
// are 2048 or 4096 quads (4-element groups): the longer one wherever it still leaves about 16
// waves of CTAs.  Measured under sustained load (60 rollouts of the large workload's launch mix
// back to back, the board at its power cap): 4096-quad chunks 16.31 ms, 2048-quad chunks 16.60 ms,
// 8192-quad chunks 16.68 ms per 28 launches of 4096 / 2048 / 1024 rows; on launches of 768 / 384 /
// 192 rows 2048-quad chunks 3.25 ms against 3.28 ms (fewer, longer CTAs drain less evenly at the
// end of a short launch).  In bursts of a few dozen launches, before the power cap bites, 2048-quad
// chunks are 1 % faster at every size: a CTA's prologue and end-of-CTA reduction cost instructions,
// and instructions cost clock once the board is power-limited.
constexpr int kRowThreads = 256;
constexpr int kRowWarps = kRowThreads / 32;
constexpr int kMinChunkQuads = 2048;                   // 8192 elements
constexpr int kMaxChunkQuads = 4096;                   // 16384 elements
constexpr long long kWantedCtas = 148LL * 4 * 16;      // CTAs for ~16 waves at 4 CTAs per SM

struct RowGeometry {
  int chunk_quads;   // quads per CTA
  int chunks;        // CTAs per row = partial sums per row
};

// Longest chunk that still leaves kWantedCtas CTAs, but never shorter than kMinChunkQuads.
inline RowGeometry row_geometry(long long rows, int elems, int forced_chunk_quads = 0) {
  const int quads = elems / 4;
  int cq = kMaxChunkQuads;
  if (forced_chunk_quads > 0) {
    cq = forced_chunk_quads;
  } else {
    while (cq > kMinChunkQuads && rows * ((quads + cq - 1) / cq) < kWantedCtas) cq >>= 1;
  }
  RowGeometry g;
  g.chunk_quads = cq;
  g.chunks = (quads + cq - 1) / cq;
  return g;
}

#ifdef __CUDACC__
// Per-row reduction in a fixed shape, without waiting on other CTAs.  Every thread of every CTA
// of the row calls this once with its warp's total (all lanes hold it).  Warp totals are
// combined through shared memory in warp order; warp 0 stores the CTA total in the CTA's fixed
// slot and takes a ticket; the CTA that draws the last ticket adds all slots in slot order
// (fp64) and hands the sum to fin(sum) on thread 0.  The result is independent of the order in
// which CTAs run.  tickets[row] is left at zero for the next launch.
template <typename Fin>
__device__ __forceinline__ void finish_row(float warp_total, int row, int chunk, int chunks,
                                           float* partials, unsigned int* tickets, Fin fin) {
  __shared__ float warp_part[kRowWarps];
  const int lane = threadIdx.x & 31;
  if (lane == 0) warp_part[threadIdx.x >> 5] = warp_total;
  __syncthreads();
  if (threadIdx.x >= 32) return;
  float v = lane < kRowWarps ? warp_part[lane] : 0.f;
  v = warp_sum(v);
  if (chunks == 1) {
    if (lane == 0) fin((double)v);
    return;
  }
  int last = 0;
  if (lane == 0) {
    partials[(size_t)row * chunks + chunk] = v;
    __threadfence();
    const unsigned int t = atomicAdd(&tickets[row], 1u);
    last = (t == (unsigned int)chunks - 1u);
  }
  last = __shfl_sync(0xFFFFFFFFu, last, 0);
  if (!last) return;
  __threadfence();
  double s = 0.0;
  for (int c = lane; c < chunks; c += 32) s += (double)__ldcg(&partials[(size_t)row * chunks + c]);
  s = warp_sum(s);
  if (lane == 0) {
    fin(s);
    tickets[row] = 0u;
  }
}

// Same reduction for NV sums per row at once (slot layout [row][chunk][NV]).
template <int NV, typename Fin>
__device__ __forceinline__ void finish_row_n(const float (&warp_total)[NV], int row, int chunk, int chunks,
                                             float* partials, unsigned int* tickets, Fin fin) {
  __shared__ float warp_part[NV][kRowWarps];
  const int lane = threadIdx.x & 31;
  if (lane == 0) {
#pragma unroll
    for (int j = 0; j < NV; ++j) warp_part[j][threadIdx.x >> 5] = warp_total[j];
  }
  __syncthreads();
  if (threadIdx.x >= 32) return;
  float v[NV];
#pragma unroll
  for (int j = 0; j < NV; ++j) v[j] = warp_sum(lane < kRowWarps ? warp_part[j][lane] : 0.f);
  double s[NV];
  if (chunks == 1) {
#pragma unroll
    for (int j = 0; j < NV; ++j) s[j] = (double)v[j];
    if (lane == 0) fin(s);
    return;
  }
  int last = 0;
  if (lane == 0) {
#pragma unroll
    for (int j = 0; j < NV; ++j) partials[((size_t)row * chunks + chunk) * NV + j] = v[j];
    __threadfence();
    const unsigned int t = atomicAdd(&tickets[row], 1u);
    last = (t == (unsigned int)chunks - 1u);
  }
  last = __shfl_sync(0xFFFFFFFFu, last, 0);
  if (!last) return;
  __threadfence();
#pragma unroll
  for (int j = 0; j < NV; ++j) {
    double a = 0.0;
    for (int c = lane; c < chunks; c += 32)
      a += (double)__ldcg(&partials[((size_t)row * chunks + c) * NV + j]);
    s[j] = warp_sum(a);
  }
  if (lane == 0) {
    fin(s);
    tickets[row] = 0u;
  }
}
#endif

// ---------------------------------------------------------------- launchers (device pointers)
struct RowScratch {
  float* partials;        // [rows * row_geometry(rows, elems).chunks * sums per row (1 or 2)]
  unsigned int* tickets;  // [rows], zero between launches
};

int launch_step(int n_rows, int elems, int vel_dtype, const float* x_in, const void* vel,
                const int32_t* src_rows, const int32_t* traj_id, float* x_out, float* logp_out,
                uint64_t seed, int32_t step, double c_x, double c_v, double noise_std,
                int logp_mean, RowScratch scratch, cudaStream_t stream, int rows_in = 0,
                int32_t* status = nullptr, float* xmean_out = nullptr);

int launch_score(int n_rows, int elems, int vel_dtype, const float* x, const void* vel,
                 double p_x, double p_v, float* scores_out, void* preview_out, int preview_bf16,
                 RowScratch scratch, cudaStream_t stream, int forced_chunk_quads = 0);

int launch_preview(int n_rows, int elems, int vel_dtype, const float* x, const void* vel, double p_x,
                   double p_v, void* out, int out_bf16, cudaStream_t stream);

int launch_policy_logprob(int n_rows, int elems, int vel_dtype, const float* x, const float* x_next,
                          const void* vel, const void* vel_ref, double c_x, double c_v,
                          double noise_std, int logp_mean, float* logp_out, float* kl_out,
                          RowScratch scratch, cudaStream_t stream);

int launch_policy_objective(int n_steps, int n_rows, const float* logp_new, const float* logp_old,
                            const float* kl, const float* adv, float clip_eps, float beta,
                            float* ratio, float* dlogp, float* objective, double* cta_part,
                            unsigned int* ticket, cudaStream_t stream);

int launch_policy_backward(int n_rows, int elems, int vel_dtype, const float* x, const float* x_next,
                           const void* vel, const void* vel_ref, double c_x, double c_v,
                           double noise_std, int logp_mean, const float* dlogp, double dkl,
                           void* grad_vel, cudaStream_t stream);

int launch_ovf(int n_groups, int n, int k, const float* scores, int32_t* keep_idx,
               int32_t* src_rows, float* sel_var, float* kept_scores, float* adv, float adv_eps,
               const int32_t* traj_in, int32_t* traj_out, int32_t* status, cudaStream_t stream);

int launch_group_stats(int n_groups, int n, const float* scores, double delta, float* mean,
                       float* std_out, float* clustered, cudaStream_t stream);

int launch_uniform_select(int n_groups, int n, int k, uint64_t seed, uint32_t stage,
                          uint32_t group_offset, int32_t* keep_idx, int32_t* src_rows,
                          const int32_t* traj_in, int32_t* traj_out, cudaStream_t stream);

int launch_advantages(int n_groups, int K, const float* rewards, float eps, float* adv,
                      float* mean, float* std_out, cudaStream_t stream);

int launch_compact(int n_groups, int n_prev, int k, const int32_t* keep_idx, const void* src,
                   void* dst, size_t row_bytes, cudaStream_t stream, int32_t* status = nullptr);

int launch_survivor_rows(int n_groups, int n_expand, int n_steps, int n_stages, const int32_t* stage_step,
                         const int32_t* stage_keep, const int32_t* keep_idx, int32_t* rows_out,
                         int32_t* status, cudaStream_t stream);

int launch_survivor_logp(const int32_t* rows, const float* logp_packed, float* logp_out,
                         const long long* step_off_dev, int n_steps, int n_final, int32_t* status,
                         cudaStream_t stream);

int launch_iota(int32_t* dst, int n, int32_t base, cudaStream_t stream);

int launch_wait_selftest(int32_t* status, cudaStream_t stream);

int launch_philox_raw(int64_t n, const uint32_t* ctr, const uint32_t* key, uint32_t* out,
                      cudaStream_t stream);

int launch_normal_rows(uint64_t seed, int32_t step, int32_t stream_id, int n_rows, int d,
                       const int32_t* traj_id, float* out, cudaStream_t stream);

}  // namespace pg
