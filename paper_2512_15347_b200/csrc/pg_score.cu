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
  int chunk_quads;
  int chunks;
  float p_x, p_v;
  double inv_d;
};

__device__ __forceinline__ float4 unpack_vel(const float4& raw) { return raw; }
__device__ __forceinline__ float4 unpack_vel(const uint2& raw) {
  float4 r;
  r.x = __uint_as_float(raw.x << 16);
  r.y = __uint_as_float(raw.x & 0xFFFF0000u);
  r.z = __uint_as_float(raw.y << 16);
  r.w = __uint_as_float(raw.y & 0xFFFF0000u);
  return r;
}
template <typename T> struct VelRaw;
template <> struct VelRaw<float> { using type = float4; };
template <> struct VelRaw<__nv_bfloat16> { using type = uint2; };

constexpr int kScoreUnroll = 4;   // quads per thread and iteration (loads of the next batch in flight)

template <typename VelT, bool kUseVel, bool kEmit>
__global__ void __launch_bounds__(kRowThreads)
score_kernel(const __grid_constant__ ScoreParams p) {
  using Raw = typename VelRaw<VelT>::type;
  const int row = blockIdx.x / p.chunks;
  const int chunk = blockIdx.x - row * p.chunks;
  const float4* x = reinterpret_cast<const float4*>(p.x) + (size_t)row * p.quads_per_row;
  const Raw* vel = reinterpret_cast<const Raw*>(p.vel) + (size_t)row * p.quads_per_row;
  float4* prev = kEmit ? reinterpret_cast<float4*>(p.preview_out) + (size_t)row * p.quads_per_row : nullptr;
  const int q_begin = chunk * p.chunk_quads;
  const int q_end = min(q_begin + p.chunk_quads, p.quads_per_row);

  float4 xv[kScoreUnroll], nx[kScoreUnroll];
  Raw vv[kScoreUnroll], nv[kScoreUnroll];
  auto load = [&](int q, float4 (&xs)[kScoreUnroll], Raw (&vs)[kScoreUnroll]) {
#pragma unroll
    for (int u = 0; u < kScoreUnroll; ++u) {
      const int qq = q + u * kRowThreads;
      if (qq < q_end) {
        xs[u] = __ldcs(x + qq);
        if (kUseVel) vs[u] = __ldcs(vel + qq);
      }
    }
  };
  float acc = 0.f;
  int q = q_begin + threadIdx.x;
  load(q, xv, vv);
  while (q < q_end) {
    const int nq = q + kScoreUnroll * kRowThreads;
    load(nq, nx, nv);
#pragma unroll
    for (int u = 0; u < kScoreUnroll; ++u) {
      const int qq = q + u * kRowThreads;
      if (qq < q_end) {
        float4 h;
        h.x = p.p_x * xv[u].x;
        h.y = p.p_x * xv[u].y;
        h.z = p.p_x * xv[u].z;
        h.w = p.p_x * xv[u].w;
        if (kUseVel) {
          const float4 vf = unpack_vel(vv[u]);
          h.x = fmaf(p.p_v, vf.x, h.x);
          h.y = fmaf(p.p_v, vf.y, h.y);
          h.z = fmaf(p.p_v, vf.z, h.z);
          h.w = fmaf(p.p_v, vf.w, h.w);
        }
        acc += (h.x + h.y) + (h.z + h.w);
        if (kEmit) __stcs(prev + qq, h);
      }
    }
#pragma unroll
    for (int u = 0; u < kScoreUnroll; ++u) { xv[u] = nx[u]; vv[u] = nv[u]; }
    q = nq;
  }

  acc = warp_sum(acc);
  finish_row(acc, row, chunk, p.chunks, p.partials, p.tickets,
             [&](double sum) { p.scores_out[row] = (float)(sum * p.inv_d); });
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
                 RowScratch scratch, cudaStream_t stream, int forced_chunk_quads) {
  if (n_rows == 0) return PG_OK;
  const RowGeometry geo = row_geometry(n_rows, elems, forced_chunk_quads);
  ScoreParams p;
  p.x = x;
  p.vel = vel;
  p.scores_out = scores_out;
  p.preview_out = preview_out;
  p.partials = scratch.partials;
  p.tickets = scratch.tickets;
  p.quads_per_row = elems / 4;
  p.chunk_quads = geo.chunk_quads;
  p.chunks = geo.chunks;
  p.p_x = (float)p_x;
  p.p_v = (float)p_v;
  p.inv_d = 1.0 / (double)elems;
  const long long blocks = (long long)n_rows * geo.chunks;
  if (blocks > 0x7FFFFFFFLL) return PG_EINVAL;
  const dim3 grid((unsigned)blocks);
  const bool use_vel = (p_v != 0.0);
  if (vel_dtype == PG_VEL_BF16) dispatch_score<__nv_bfloat16>(p, use_vel, preview_out != nullptr, grid, stream);
  else                          dispatch_score<float>(p, use_vel, preview_out != nullptr, grid, stream);
  PG_LAUNCH_CHECK();
  return PG_OK;
}

}  // namespace pg
