// ODE look-ahead preview and latent score (Eq. "ode_lookahead_method", Eq. "proxy_reward_method"):
// x_hat = p_x * x + p_v * v, score = mean over the elements of x_hat.  Read-only streaming pass,
// optionally emitting x_hat in the same pass as fp32 or as bf16 (what a decoder + reward model
// placed between preview and selection consume: 8 bytes per element for score and preview
// together instead of a 6-byte scoring pass plus an 8-byte emission pass); the per-trajectory sum
// uses the same fixed-shape reduction as the step kernel, so scores are reproducible from run
// to run.  The score is always reduced from the fp32 preview, whatever is emitted.
#include "pg_common.cuh"

namespace pg {

struct ScoreParams {
  const float* x;
  const void* vel;
  float* scores_out;
  void* preview_out;
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

__device__ __forceinline__ void store_preview(float* out, size_t quad, const float4& v) {
  __stcs(reinterpret_cast<float4*>(out) + quad, v);
}
__device__ __forceinline__ void store_preview(__nv_bfloat16* out, size_t quad, const float4& v) {
  const __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y);
  const __nv_bfloat162 hi = __floats2bfloat162_rn(v.z, v.w);
  uint2 w;
  w.x = *reinterpret_cast<const unsigned int*>(&lo);
  w.y = *reinterpret_cast<const unsigned int*>(&hi);
  __stcs(reinterpret_cast<uint2*>(out) + quad, w);
}

// What the scoring pass writes besides the scores.
enum : int { kEmitNone = 0, kEmitF32 = 1, kEmitBf16 = 2 };
template <int kEmit> struct EmitType { using type = float; };
template <> struct EmitType<kEmitBf16> { using type = __nv_bfloat16; };

constexpr int kScoreUnroll = 4;   // quads per thread and iteration (loads of the next batch in flight)

// The bf16-prediction variants that also write the preview are held to 64 registers (four CTAs per SM, like the
// scoring-only variants): at the 69 - 70 registers the compiler would otherwise take, three CTAs
// fit and the bf16-emitting pass measured 6.47 instead of 6.82 TB/s on 2048 rows of 262144.
// kReduce = false: emission only (pg_preview): the same streaming loop without the row reduction.
template <typename VelT, bool kUseVel, int kEmit, bool kReduce = true>
__global__ void __launch_bounds__(kRowThreads, (kEmit != kEmitNone && sizeof(VelT) == 2) ? 4 : 0)
score_kernel(const __grid_constant__ ScoreParams p) {
  using Raw = typename VelRaw<VelT>::type;
  using OutT = typename EmitType<kEmit>::type;
  const int row = blockIdx.x / p.chunks;
  const int chunk = blockIdx.x - row * p.chunks;
  const float4* x = reinterpret_cast<const float4*>(p.x) + (size_t)row * p.quads_per_row;
  const Raw* vel = reinterpret_cast<const Raw*>(p.vel) + (size_t)row * p.quads_per_row;
  OutT* prev = kEmit ? reinterpret_cast<OutT*>(p.preview_out) + (size_t)row * p.quads_per_row * 4 : nullptr;
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
        if (kReduce) acc += (h.x + h.y) + (h.z + h.w);
        if (kEmit) store_preview(prev, (size_t)qq, h);
      }
    }
#pragma unroll
    for (int u = 0; u < kScoreUnroll; ++u) { xv[u] = nx[u]; vv[u] = nv[u]; }
    q = nq;
  }

  if (!kReduce) return;
  acc = warp_sum(acc);
  finish_row(acc, row, chunk, p.chunks, p.partials, p.tickets,
             [&](double sum) { p.scores_out[row] = (float)(sum * p.inv_d); });
}

template <typename VelT, bool kUseVel>
static void dispatch_score_emit(const ScoreParams& p, int emit, dim3 grid, cudaStream_t stream) {
  const dim3 block(kRowThreads);
  if (emit == kEmitBf16)     score_kernel<VelT, kUseVel, kEmitBf16><<<grid, block, 0, stream>>>(p);
  else if (emit == kEmitF32) score_kernel<VelT, kUseVel, kEmitF32><<<grid, block, 0, stream>>>(p);
  else                       score_kernel<VelT, kUseVel, kEmitNone><<<grid, block, 0, stream>>>(p);
}

template <typename VelT>
static void dispatch_score(const ScoreParams& p, bool use_vel, int emit, dim3 grid,
                           cudaStream_t stream) {
  if (use_vel) dispatch_score_emit<VelT, true>(p, emit, grid, stream);
  else         dispatch_score_emit<VelT, false>(p, emit, grid, stream);
}

int launch_score(int n_rows, int elems, int vel_dtype, const float* x, const void* vel,
                 double p_x, double p_v, float* scores_out, void* preview_out, int preview_bf16,
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
  const int emit = !preview_out ? kEmitNone : (preview_bf16 ? kEmitBf16 : kEmitF32);
  if (vel_dtype == PG_VEL_BF16) dispatch_score<__nv_bfloat16>(p, use_vel, emit, grid, stream);
  else                          dispatch_score<float>(p, use_vel, emit, grid, stream);
  PG_LAUNCH_CHECK();
  return PG_OK;
}

// ---------------------------------------------------------------- preview emission only

// x_hat = p_x x + p_v v written in fp32 or bf16 (for a decoder that follows); no reduction.
int launch_preview(int n_rows, int elems, int vel_dtype, const float* x, const void* vel, double p_x,
                   double p_v, void* out, int out_bf16, cudaStream_t stream) {
  if (n_rows == 0) return PG_OK;
  const RowGeometry geo = row_geometry(n_rows, elems);
  ScoreParams p;
  p.x = x;
  p.vel = vel;
  p.scores_out = nullptr;
  p.preview_out = out;
  p.partials = nullptr;
  p.tickets = nullptr;
  p.quads_per_row = elems / 4;
  p.chunk_quads = geo.chunk_quads;
  p.chunks = geo.chunks;
  p.p_x = (float)p_x;
  p.p_v = (float)p_v;
  p.inv_d = 0.0;
  const long long blocks = (long long)n_rows * geo.chunks;
  if (blocks > 0x7FFFFFFFLL) return PG_EINVAL;
  const dim3 grid((unsigned)blocks), block(kRowThreads);
  if (vel_dtype == PG_VEL_BF16) {
    if (out_bf16) score_kernel<__nv_bfloat16, true, kEmitBf16, false><<<grid, block, 0, stream>>>(p);
    else          score_kernel<__nv_bfloat16, true, kEmitF32, false><<<grid, block, 0, stream>>>(p);
  } else {
    if (out_bf16) score_kernel<float, true, kEmitBf16, false><<<grid, block, 0, stream>>>(p);
    else          score_kernel<float, true, kEmitF32, false><<<grid, block, 0, stream>>>(p);
  }
  PG_LAUNCH_CHECK();
  return PG_OK;
}

}  // namespace pg
