// ODE look-ahead preview and latent score (Eq. "ode_lookahead_method", Eq. "proxy_reward_method"):
// x_hat = p_x * x + p_v * v, score = mean over the elements of x_hat.  Read-only streaming pass
// (optionally emitting x_hat); the per-trajectory sum uses the same fixed-shape reduction as the
// step kernel, so scores are reproducible from run to run.
#include "pg_common.cuh"

namespace pg {

struct ScoreParams {
  const float* x;
  const void* vel;
  float* scores_out;
  float* preview_out;
  float* partials;
  unsigned int* tickets;
  int quads_per_row;
  int chunks;
  float p_x, p_v;
  double inv_d;
};

__device__ __forceinline__ float4 score_vel4(const float* v, size_t quad) {
  return __ldcs(reinterpret_cast<const float4*>(v) + quad);
}
__device__ __forceinline__ float4 score_vel4(const __nv_bfloat16* v, size_t quad) {
  const uint2 w = __ldcs(reinterpret_cast<const uint2*>(v) + quad);
  float4 r;
  r.x = __uint_as_float(w.x << 16);
  r.y = __uint_as_float(w.x & 0xFFFF0000u);
  r.z = __uint_as_float(w.y << 16);
  r.w = __uint_as_float(w.y & 0xFFFF0000u);
  return r;
}

template <typename VelT, bool kUseVel, bool kEmit>
__global__ void __launch_bounds__(kRowThreads)
score_kernel(const __grid_constant__ ScoreParams p) {
  const int row = blockIdx.x / p.chunks;
  const int chunk = blockIdx.x - row * p.chunks;
  const size_t base = (size_t)row * p.quads_per_row;
  const VelT* vel = reinterpret_cast<const VelT*>(p.vel);
  const int q0 = chunk * kChunkQuads + threadIdx.x;

  float4 xv[kQuadsPerThread], vv[kQuadsPerThread];
#pragma unroll
  for (int u = 0; u < kQuadsPerThread; ++u) {
    const int q = q0 + u * kRowThreads;
    if (q < p.quads_per_row) {
      xv[u] = __ldcs(reinterpret_cast<const float4*>(p.x) + base + q);
      if (kUseVel) vv[u] = score_vel4(vel, base + q);
    }
  }
  float acc = 0.f;
#pragma unroll
  for (int u = 0; u < kQuadsPerThread; ++u) {
    const int q = q0 + u * kRowThreads;
    if (q < p.quads_per_row) {
      float4 h;
      h.x = p.p_x * xv[u].x;
      h.y = p.p_x * xv[u].y;
      h.z = p.p_x * xv[u].z;
      h.w = p.p_x * xv[u].w;
      if (kUseVel) {
        h.x = fmaf(p.p_v, vv[u].x, h.x);
        h.y = fmaf(p.p_v, vv[u].y, h.y);
        h.z = fmaf(p.p_v, vv[u].z, h.z);
        h.w = fmaf(p.p_v, vv[u].w, h.w);
      }
      acc += (h.x + h.y) + (h.z + h.w);
      if (kEmit) __stcs(reinterpret_cast<float4*>(p.preview_out) + base + q, h);
    }
  }

  __shared__ float warp_part[kRowThreads / 32];
  __shared__ bool is_last;
  acc = warp_sum(acc);
  if ((threadIdx.x & 31) == 0) warp_part[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x < 32) {
    float v = (threadIdx.x < kRowThreads / 32) ? warp_part[threadIdx.x] : 0.f;
    v = warp_sum(v);
    if (threadIdx.x == 0) {
      if (p.chunks == 1) {
        p.scores_out[row] = (float)((double)v * p.inv_d);
        is_last = false;
      } else {
        p.partials[(size_t)row * p.chunks + chunk] = v;
        __threadfence();
        const unsigned int t = atomicAdd(&p.tickets[row], 1u);
        is_last = (t == (unsigned int)p.chunks - 1u);
      }
    }
  }
  __syncthreads();
  if (!is_last) return;
  if (threadIdx.x < 32) {
    __threadfence();
    double s = 0.0;
    for (int c = threadIdx.x; c < p.chunks; c += 32)
      s += (double)__ldcg(&p.partials[(size_t)row * p.chunks + c]);
    s = warp_sum(s);
    if (threadIdx.x == 0) {
      p.scores_out[row] = (float)(s * p.inv_d);
      p.tickets[row] = 0u;
    }
  }
}

template <typename VelT>
static void dispatch_score(const ScoreParams& p, bool use_vel, bool emit, dim3 grid,
                           cudaStream_t stream) {
  const dim3 block(kRowThreads);
  if (use_vel) {
    if (emit) score_kernel<VelT, true, true><<<grid, block, 0, stream>>>(p);
    else      score_kernel<VelT, true, false><<<grid, block, 0, stream>>>(p);
  } else {
    if (emit) score_kernel<VelT, false, true><<<grid, block, 0, stream>>>(p);
    else      score_kernel<VelT, false, false><<<grid, block, 0, stream>>>(p);
  }
}

int launch_score(int n_rows, int elems, int vel_dtype, const float* x, const void* vel,
                 double p_x, double p_v, float* scores_out, float* preview_out,
                 RowScratch scratch, cudaStream_t stream) {
  if (n_rows == 0) return PG_OK;
  ScoreParams p;
  p.x = x;
  p.vel = vel;
  p.scores_out = scores_out;
  p.preview_out = preview_out;
  p.partials = scratch.partials;
  p.tickets = scratch.tickets;
  p.quads_per_row = elems / 4;
  p.chunks = chunks_per_row(elems);
  p.p_x = (float)p_x;
  p.p_v = (float)p_v;
  p.inv_d = 1.0 / (double)elems;
  const long long blocks = (long long)n_rows * p.chunks;
  if (blocks > 0x7FFFFFFFLL) return PG_EINVAL;
  const dim3 grid((unsigned)blocks);
  const bool use_vel = (p_v != 0.0);
  if (vel_dtype == PG_VEL_BF16) dispatch_score<__nv_bfloat16>(p, use_vel, preview_out != nullptr, grid, stream);
  else                          dispatch_score<float>(p, use_vel, preview_out != nullptr, grid, stream);
  PG_LAUNCH_CHECK();
  return PG_OK;
}

}  // namespace pg
