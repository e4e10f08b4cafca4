// Policy update on the survivors (Eq. "ratio_method", Eq. "pro_grpo_method"): log-density of
// the stored transitions under a new prediction with the Gaussian KL to a reference
// prediction (read-only streaming pass, two sums per trajectory), the clipped surrogate
// objective with dJ/dlogp, and the elementwise gradient with respect to the prediction.
#include "pg_common.cuh"

namespace pg {

__device__ __forceinline__ float4 pol_unpack(const float4& raw) { return raw; }
__device__ __forceinline__ float4 pol_unpack(const uint2& raw) {
  float4 r;
  r.x = __uint_as_float(raw.x << 16);
  r.y = __uint_as_float(raw.x & 0xFFFF0000u);
  r.z = __uint_as_float(raw.y << 16);
  r.w = __uint_as_float(raw.y & 0xFFFF0000u);
  return r;
}
template <typename T> struct PolRaw;
template <> struct PolRaw<float> { using type = float4; };
template <> struct PolRaw<__nv_bfloat16> { using type = uint2; };

// ---------------------------------------------------------------- log pi_theta and KL

struct PolicyLogpParams {
  const float* x;
  const float* x_next;
  const void* vel;
  const void* vel_ref;
  float* logp_out;
  float* kl_out;
  float* partials;
  unsigned int* tickets;
  int quads_per_row, chunk_quads, chunks;
  float c_x, c_v, inv_s;
  double logp_const;    // d/2 ln(2 pi s^2)
  double scale;         // 1 or 1/d
  double kl_scale;      // 1 / (2 s^2)
};

constexpr int kPolicyUnroll = 2;

template <typename VelT, bool kRef>
__global__ void __launch_bounds__(kRowThreads)
policy_logprob_kernel(const __grid_constant__ PolicyLogpParams p) {
  using Raw = typename PolRaw<VelT>::type;
  const int row = blockIdx.x / p.chunks;
  const int chunk = blockIdx.x - row * p.chunks;
  const size_t base = (size_t)row * p.quads_per_row;
  const float4* __restrict__ x = reinterpret_cast<const float4*>(p.x) + base;
  const float4* __restrict__ xn = reinterpret_cast<const float4*>(p.x_next) + base;
  const Raw* __restrict__ vel = reinterpret_cast<const Raw*>(p.vel) + base;
  const Raw* __restrict__ ref = kRef ? reinterpret_cast<const Raw*>(p.vel_ref) + base : nullptr;
  const int q_begin = chunk * p.chunk_quads;
  const int q_end = min(q_begin + p.chunk_quads, p.quads_per_row);

  float4 xv[kPolicyUnroll], nv[kPolicyUnroll], xv2[kPolicyUnroll], nv2[kPolicyUnroll];
  Raw vv[kPolicyUnroll], rv[kPolicyUnroll], vv2[kPolicyUnroll], rv2[kPolicyUnroll];
  auto load = [&](int q, float4 (&a)[kPolicyUnroll], float4 (&b)[kPolicyUnroll],
                  Raw (&c)[kPolicyUnroll], Raw (&d)[kPolicyUnroll]) {
#pragma unroll
    for (int u = 0; u < kPolicyUnroll; ++u) {
      const int qq = q + u * kRowThreads;
      if (qq < q_end) {
        a[u] = __ldcs(x + qq);
        b[u] = __ldcs(xn + qq);
        c[u] = __ldcs(vel + qq);
        if (kRef) d[u] = __ldcs(ref + qq);
      }
    }
  };
  float acc[2] = {0.f, 0.f};
  int q = q_begin + threadIdx.x;
  load(q, xv, nv, vv, rv);
  while (q < q_end) {
    const int nq = q + kPolicyUnroll * kRowThreads;
    load(nq, xv2, nv2, vv2, rv2);
#pragma unroll
    for (int u = 0; u < kPolicyUnroll; ++u) {
      if (q + u * kRowThreads < q_end) {
        const float4 vf = pol_unpack(vv[u]);
        const float zx = (nv[u].x - fmaf(p.c_v, vf.x, p.c_x * xv[u].x)) * p.inv_s;
        const float zy = (nv[u].y - fmaf(p.c_v, vf.y, p.c_x * xv[u].y)) * p.inv_s;
        const float zz = (nv[u].z - fmaf(p.c_v, vf.z, p.c_x * xv[u].z)) * p.inv_s;
        const float zw = (nv[u].w - fmaf(p.c_v, vf.w, p.c_x * xv[u].w)) * p.inv_s;
        acc[0] += (zx * zx + zy * zy) + (zz * zz + zw * zw);
        if (kRef) {
          const float4 rf = pol_unpack(rv[u]);
          const float dx = p.c_v * (vf.x - rf.x), dy = p.c_v * (vf.y - rf.y);
          const float dz = p.c_v * (vf.z - rf.z), dw = p.c_v * (vf.w - rf.w);
          acc[1] += (dx * dx + dy * dy) + (dz * dz + dw * dw);
        }
      }
    }
#pragma unroll
    for (int u = 0; u < kPolicyUnroll; ++u) { xv[u] = xv2[u]; nv[u] = nv2[u]; vv[u] = vv2[u]; rv[u] = rv2[u]; }
    q = nq;
  }
  acc[0] = warp_sum(acc[0]);
  acc[1] = warp_sum(acc[1]);
  float* logp_out = p.logp_out;
  float* kl_out = p.kl_out;
  const double lc = p.logp_const, sc = p.scale, ks = p.kl_scale;
  finish_row_n<2>(acc, row, chunk, p.chunks, p.partials, p.tickets, [=](const double (&s)[2]) {
    logp_out[row] = (float)((-0.5 * s[0] - lc) * sc);
    if (kRef) kl_out[row] = (float)(s[1] * ks * sc);
  });
}

int launch_policy_logprob(int n_rows, int elems, int vel_dtype, const float* x, const float* x_next,
                          const void* vel, const void* vel_ref, double c_x, double c_v,
                          double noise_std, int logp_mean, float* logp_out, float* kl_out,
                          RowScratch scratch, cudaStream_t stream) {
  if (n_rows == 0) return PG_OK;
  const RowGeometry geo = row_geometry(n_rows, elems);
  PolicyLogpParams p;
  p.x = x; p.x_next = x_next; p.vel = vel; p.vel_ref = vel_ref;
  p.logp_out = logp_out; p.kl_out = kl_out;
  p.partials = scratch.partials; p.tickets = scratch.tickets;
  p.quads_per_row = elems / 4; p.chunk_quads = geo.chunk_quads; p.chunks = geo.chunks;
  p.c_x = (float)c_x; p.c_v = (float)c_v; p.inv_s = (float)(1.0 / noise_std);
  const double two_pi = 6.283185307179586476925286766559;
  p.logp_const = 0.5 * (double)elems * log(two_pi * noise_std * noise_std);
  p.scale = logp_mean ? 1.0 / (double)elems : 1.0;
  p.kl_scale = 1.0 / (2.0 * noise_std * noise_std);
  const long long blocks = (long long)n_rows * geo.chunks;
  if (blocks > 0x7FFFFFFFLL) return PG_EINVAL;
  const dim3 grid((unsigned)blocks), block(kRowThreads);
  const bool has_ref = vel_ref != nullptr;
  if (vel_dtype == PG_VEL_BF16) {
    if (has_ref) policy_logprob_kernel<__nv_bfloat16, true><<<grid, block, 0, stream>>>(p);
    else         policy_logprob_kernel<__nv_bfloat16, false><<<grid, block, 0, stream>>>(p);
  } else {
    if (has_ref) policy_logprob_kernel<float, true><<<grid, block, 0, stream>>>(p);
    else         policy_logprob_kernel<float, false><<<grid, block, 0, stream>>>(p);
  }
  PG_LAUNCH_CHECK();
  return PG_OK;
}

// ---------------------------------------------------------------- clipped surrogate objective

constexpr int kObjThreads = 1024;
constexpr int kObjMinEntries = 8 * kObjThreads;      // entries per CTA: at least eight per thread

// Ratios, clipped surrogate, dJ/dlogp for all (step, trajectory) pairs and the mean objective.
// CTA b handles the entries [b * per_cta, (b + 1) * per_cta): every thread sums its entries in
// index order, the CTA combines them in a fixed tree (fp64) and stores its partial sum in slot b;
// the CTA that draws the last ticket adds the slots in slot order.  The split depends only on
// the number of entries, so the objective is the same bits on every run.
__global__ void __launch_bounds__(kObjThreads)
policy_objective_kernel(int n_steps, int n_rows, long long per_cta, const float* logp_new,
                        const float* logp_old, const float* kl, const float* adv, float clip_eps,
                        float beta, float* ratio, float* dlogp, float* objective, double* cta_part,
                        unsigned int* ticket) {
  __shared__ double part[kObjThreads / 32];
  __shared__ int is_last;
  const long long total = (long long)n_steps * n_rows;
  const double inv = 1.0 / (double)total;
  const double lo = 1.0 - (double)clip_eps, hi = 1.0 + (double)clip_eps;
  const long long begin = (long long)blockIdx.x * per_cta;
  const long long end = begin + per_cta < total ? begin + per_cta : total;
  double acc = 0.0;
  for (long long j = begin + threadIdx.x; j < end; j += kObjThreads) {
    const int i = (int)(j % n_rows);
    const double r = exp((double)logp_new[j] - (double)logp_old[j]);
    const double rc = r < lo ? lo : (r > hi ? hi : r);
    const double a = (double)adv[i];
    const double s1 = r * a, s2 = rc * a;
    acc += (s1 < s2 ? s1 : s2) - (kl ? (double)beta * (double)kl[j] : 0.0);
    if (ratio) ratio[j] = (float)r;
    dlogp[j] = (s1 <= s2) ? (float)(inv * a * r) : 0.f;
  }
  acc = warp_sum(acc);
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = acc;
  __syncthreads();
  double v = 0.0;
  if (threadIdx.x < 32) v = warp_sum(part[threadIdx.x]);
  if (gridDim.x == 1) {
    if (threadIdx.x == 0) objective[0] = (float)(v * inv);
    return;
  }
  if (threadIdx.x == 0) {
    cta_part[blockIdx.x] = v;
    __threadfence();
    is_last = atomicAdd(ticket, 1u) == gridDim.x - 1u;
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  // slots in slot order: thread t takes slot t (at most kObjThreads slots), then the same tree
  double s = threadIdx.x < gridDim.x ? __ldcg(cta_part + threadIdx.x) : 0.0;
  s = warp_sum(s);
  __syncthreads();                       // part[] is reused
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = s;
  __syncthreads();
  if (threadIdx.x < 32) {
    const double w = warp_sum(part[threadIdx.x]);
    if (threadIdx.x == 0) {
      objective[0] = (float)(w * inv);
      *ticket = 0u;                      // ready for the next launch
    }
  }
}

int launch_policy_objective(int n_steps, int n_rows, const float* logp_new, const float* logp_old,
                            const float* kl, const float* adv, float clip_eps, float beta,
                            float* ratio, float* dlogp, float* objective, double* cta_part,
                            unsigned int* ticket, cudaStream_t stream) {
  const long long total = (long long)n_steps * n_rows;
  if (total == 0) return PG_OK;
  // entries per CTA: kObjMinEntries, or more (a multiple of the CTA size) so that kObjThreads slots suffice
  long long per_cta = kObjMinEntries;
  if ((total + per_cta - 1) / per_cta > kObjThreads) {
    per_cta = (total + kObjThreads - 1) / kObjThreads;
    per_cta = (per_cta + kObjThreads - 1) / kObjThreads * kObjThreads;
  }
  const unsigned int ctas = (unsigned int)((total + per_cta - 1) / per_cta);
  policy_objective_kernel<<<ctas, kObjThreads, 0, stream>>>(n_steps, n_rows, per_cta, logp_new, logp_old, kl,
                                                            adv, clip_eps, beta, ratio, dlogp, objective,
                                                            cta_part, ticket);
  PG_LAUNCH_CHECK();
  return PG_OK;
}

// ---------------------------------------------------------------- gradient w.r.t. the prediction

struct PolicyBwdParams {
  const float* x;
  const float* x_next;
  const void* vel;
  const void* vel_ref;
  const float* dlogp;
  void* grad;
  int quads_per_row, chunk_quads, chunks;
  float c_x, c_v;
  float lp_coef;     // c_v / s^2 (/ d)
  float kl_coef;     // dkl * c_v^2 / s^2 (/ d)
};

__device__ __forceinline__ void store_grad(float* g, size_t quad, const float4& v) {
  __stcs(reinterpret_cast<float4*>(g) + quad, v);
}
__device__ __forceinline__ void store_grad(__nv_bfloat16* g, size_t quad, const float4& v) {
  const __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y);
  const __nv_bfloat162 hi = __floats2bfloat162_rn(v.z, v.w);
  uint2 w;
  w.x = *reinterpret_cast<const unsigned int*>(&lo);
  w.y = *reinterpret_cast<const unsigned int*>(&hi);
  __stcs(reinterpret_cast<uint2*>(g) + quad, w);
}

template <typename VelT, bool kRef>
__global__ void __launch_bounds__(kRowThreads)
policy_backward_kernel(const __grid_constant__ PolicyBwdParams p) {
  using Raw = typename PolRaw<VelT>::type;
  const int row = blockIdx.x / p.chunks;
  const int chunk = blockIdx.x - row * p.chunks;
  const size_t base = (size_t)row * p.quads_per_row;
  const float4* __restrict__ x = reinterpret_cast<const float4*>(p.x) + base;
  const float4* __restrict__ xn = reinterpret_cast<const float4*>(p.x_next) + base;
  const Raw* __restrict__ vel = reinterpret_cast<const Raw*>(p.vel) + base;
  const Raw* __restrict__ ref = kRef ? reinterpret_cast<const Raw*>(p.vel_ref) + base : nullptr;
  VelT* grad = reinterpret_cast<VelT*>(p.grad);
  const float a = p.dlogp[row] * p.lp_coef;
  const float b = p.kl_coef;
  const int q_begin = chunk * p.chunk_quads;
  const int q_end = min(q_begin + p.chunk_quads, p.quads_per_row);
  constexpr int kU = 4;
  for (int q0 = q_begin + threadIdx.x; q0 < q_end; q0 += kU * kRowThreads) {
    float4 xv[kU], nv[kU];
    Raw vv[kU], rv[kU];
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      const int q = q0 + u * kRowThreads;
      if (q < q_end) {
        xv[u] = __ldcs(x + q);
        nv[u] = __ldcs(xn + q);
        vv[u] = __ldcs(vel + q);
        if (kRef) rv[u] = __ldcs(ref + q);
      }
    }
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      const int q = q0 + u * kRowThreads;
      if (q < q_end) {
        const float4 vf = pol_unpack(vv[u]);
        float4 g;
        g.x = a * (nv[u].x - fmaf(p.c_v, vf.x, p.c_x * xv[u].x));
        g.y = a * (nv[u].y - fmaf(p.c_v, vf.y, p.c_x * xv[u].y));
        g.z = a * (nv[u].z - fmaf(p.c_v, vf.z, p.c_x * xv[u].z));
        g.w = a * (nv[u].w - fmaf(p.c_v, vf.w, p.c_x * xv[u].w));
        if (kRef) {
          const float4 rf = pol_unpack(rv[u]);
          g.x = fmaf(b, vf.x - rf.x, g.x);
          g.y = fmaf(b, vf.y - rf.y, g.y);
          g.z = fmaf(b, vf.z - rf.z, g.z);
          g.w = fmaf(b, vf.w - rf.w, g.w);
        }
        store_grad(grad, base + q, g);
      }
    }
  }
}

int launch_policy_backward(int n_rows, int elems, int vel_dtype, const float* x, const float* x_next,
                           const void* vel, const void* vel_ref, double c_x, double c_v,
                           double noise_std, int logp_mean, const float* dlogp, double dkl,
                           void* grad_vel, cudaStream_t stream) {
  if (n_rows == 0) return PG_OK;
  const RowGeometry geo = row_geometry(n_rows, elems);
  PolicyBwdParams p;
  p.x = x; p.x_next = x_next; p.vel = vel; p.vel_ref = vel_ref; p.dlogp = dlogp; p.grad = grad_vel;
  p.quads_per_row = elems / 4; p.chunk_quads = geo.chunk_quads; p.chunks = geo.chunks;
  p.c_x = (float)c_x; p.c_v = (float)c_v;
  const double scale = logp_mean ? 1.0 / (double)elems : 1.0;
  const double inv_s2 = 1.0 / (noise_std * noise_std);
  p.lp_coef = (float)(c_v * inv_s2 * scale);
  p.kl_coef = (float)(dkl * c_v * c_v * inv_s2 * scale);
  const long long blocks = (long long)n_rows * geo.chunks;
  if (blocks > 0x7FFFFFFFLL) return PG_EINVAL;
  const dim3 grid((unsigned)blocks), block(kRowThreads);
  const bool has_ref = vel_ref != nullptr;
  if (vel_dtype == PG_VEL_BF16) {
    if (has_ref) policy_backward_kernel<__nv_bfloat16, true><<<grid, block, 0, stream>>>(p);
    else         policy_backward_kernel<__nv_bfloat16, false><<<grid, block, 0, stream>>>(p);
  } else {
    if (has_ref) policy_backward_kernel<float, true><<<grid, block, 0, stream>>>(p);
    else         policy_backward_kernel<float, false><<<grid, block, 0, stream>>>(p);
  }
  PG_LAUNCH_CHECK();
  return PG_OK;
}

}  // namespace pg
