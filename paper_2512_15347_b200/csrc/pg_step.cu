// Fused Euler-Maruyama step + Gaussian policy log-probability (Eq. "euler_method").
//
// One CTA streams one chunk of one trajectory: x and the prediction are read once with
// 128/64-bit coalesced loads, the loads of the next pair of quads being issued before the
// current pair is computed (full chunks alternate between two register sets without bounds
// checks); the noise is generated in registers (one Philox block per 4 elements); x' is written
// once.  Sum of squared noise: for a Box-Muller pair a^2 + b^2 equals -2 ln u1, so the radius
// term (as log2 u1, scaled once per thread) is accumulated directly.  The per-trajectory sum is reduced thread -> warp (shuffle) ->
// CTA (shared memory) -> trajectory (fixed-slot partials finished by the last-arriving CTA,
// without waiting), so the result does not depend on scheduling.
#include "pg_common.cuh"

namespace pg {

struct StepParams {
  const float* x_in;
  const void* vel;
  const int32_t* src_rows;
  const int32_t* traj_id;
  float* x_out;
  float* logp_out;
  float* xmean_out;       // [rows] mean of x_out per row, or null
  float* partials;
  unsigned int* tickets;
  int32_t* status;        // device status word (bit 2: gather index out of range) or null
  int rows_in;            // rows of x_in / vel that src_rows may address
  int quads_per_row;      // d / 4
  int chunk_quads;        // quads per CTA
  int chunks;             // CTAs per row
  int chunk_shift;        // log2(chunks) when chunks is a power of two, else -1
  uint32_t step;
  float c_x, c_v;
  float neg_scale2;       // -2 ln 2 * noise_std^2: log2(u1) times this is (noise_std * radius)^2
  double logp_const;      // d/2 * ln(2 pi noise_std^2)
  double logp_scale;      // 1 or 1/d
  double inv_d;           // 1/d
  PhiloxKeys rk;
};

struct VelF32 { float4 raw; };
struct VelBf16 { uint2 raw; };

__device__ __forceinline__ void load_vel(const float* v, size_t quad, VelF32& out) {
  out.raw = __ldcs(reinterpret_cast<const float4*>(v) + quad);
}
__device__ __forceinline__ void load_vel(const __nv_bfloat16* v, size_t quad, VelBf16& out) {
  out.raw = __ldcs(reinterpret_cast<const uint2*>(v) + quad);
}
__device__ __forceinline__ float4 vel_f32(const VelF32& v) { return v.raw; }
__device__ __forceinline__ float4 vel_f32(const VelBf16& v) {
  float4 r;
  r.x = __uint_as_float(v.raw.x << 16);
  r.y = __uint_as_float(v.raw.x & 0xFFFF0000u);
  r.z = __uint_as_float(v.raw.y << 16);
  r.w = __uint_as_float(v.raw.y & 0xFFFF0000u);
  return r;
}
template <typename T> struct VelReg;
template <> struct VelReg<float> { using type = VelF32; };
template <> struct VelReg<__nv_bfloat16> { using type = VelBf16; };

#ifndef PG_STEP_UNROLL
#define PG_STEP_UNROLL 2       // quads per thread and loop iteration (the next batch is in flight)
#endif
#ifndef PG_STEP_MIN_CTAS
#define PG_STEP_MIN_CTAS 5     // __launch_bounds__ minimum resident CTAs per SM (bf16 prediction)
#endif
// fp32 predictions keep twice the prediction registers in flight, and the variant that also reduces
// the row means one more accumulator: one CTA less per SM, no spills
template <typename VelT, bool kNoise, bool kMean> struct StepMinCtas {
  static constexpr int value = (sizeof(VelT) == 2 && kNoise && !kMean) ? PG_STEP_MIN_CTAS : 4;
};
constexpr int kStepUnroll = PG_STEP_UNROLL;
static_assert(kMinChunkQuads % (2 * kStepUnroll * kRowThreads) == 0 && kMaxChunkQuads % kMinChunkQuads == 0,
              "full chunks must hold an even number of batches");

// One quad: mean of the transition, noise, store, radius-term accumulation.
template <bool kNoise, bool kUnitCx, bool kMean>
__device__ __forceinline__ void step_quad(const StepParams& p, uint32_t traj, int q, const float4& xv,
                                          const float4& vv, float4* __restrict__ xout, float& acc,
                                          float& acc_x) {
  float4 m;
  if (kUnitCx) {
    m.x = fmaf(p.c_v, vv.x, xv.x);
    m.y = fmaf(p.c_v, vv.y, xv.y);
    m.z = fmaf(p.c_v, vv.z, xv.z);
    m.w = fmaf(p.c_v, vv.w, xv.w);
  } else {
    m.x = fmaf(p.c_v, vv.x, p.c_x * xv.x);
    m.y = fmaf(p.c_v, vv.y, p.c_x * xv.y);
    m.z = fmaf(p.c_v, vv.z, p.c_x * xv.z);
    m.w = fmaf(p.c_v, vv.w, p.c_x * xv.w);
  }
  if (kNoise) {
    const uint4 r = philox4x32_10((uint32_t)q, p.step, traj, 0u, p.rk);
    // noise_std * xi = -(noise_std * radius) * (cos, sin): the scale enters under the square root
    float ra, ca, sa, rb, cb, sb;
    acc += box_muller(r.x, r.y, p.neg_scale2, ra, ca, sa);       // acc collects log2(u1) <= 0
    acc += box_muller(r.z, r.w, p.neg_scale2, rb, cb, sb);
    m.x = fmaf(-ra, ca, m.x);
    m.y = fmaf(-ra, sa, m.y);
    m.z = fmaf(-rb, cb, m.z);
    m.w = fmaf(-rb, sb, m.w);
  }
  if (kMean) acc_x += (m.x + m.y) + (m.z + m.w);
  __stcs(xout + q, m);
}

// kNoise: noise_std > 0.  kUnitCx: c_x == 1 (drift = prediction), one FMA per element less.
// kMean: also reduce the mean of every updated latent (the stand-in reward of the final latent,
// taken from the registers that hold x' instead of reading x' back in a pass of its own).
template <typename VelT, bool kNoise, bool kUnitCx, bool kMean>
__global__ void __launch_bounds__(kRowThreads, StepMinCtas<VelT, kNoise, kMean>::value)
step_kernel(const __grid_constant__ StepParams p) {
  using VReg = typename VelReg<VelT>::type;
  // chunks per row is a power of two for the usual latent sizes: a shift instead of a division
  const int row = p.chunk_shift >= 0 ? (int)(blockIdx.x >> p.chunk_shift) : (int)(blockIdx.x / p.chunks);
  const int chunk = blockIdx.x - row * p.chunks;
  int src = p.src_rows ? p.src_rows[row] : row;
  if ((unsigned int)src >= (unsigned int)p.rows_in) {
    // a gather index outside the input: never dereferenced; the row is computed from row 0 so
    // that the reduction protocol stays complete, and the status word reports it
    if (threadIdx.x == 0 && chunk == 0 && p.status) atomicOr(p.status, 4);
    src = 0;
  }
  const uint32_t traj = (uint32_t)p.traj_id[row];

  const float4* __restrict__ xin = reinterpret_cast<const float4*>(p.x_in) + (size_t)src * p.quads_per_row;
  const VelT* __restrict__ vel = reinterpret_cast<const VelT*>(p.vel) + (size_t)src * p.quads_per_row * 4;
  float4* __restrict__ xout = reinterpret_cast<float4*>(p.x_out) + (size_t)row * p.quads_per_row;
  const int q_begin = chunk * p.chunk_quads;
  const int q_end = min(q_begin + p.chunk_quads, p.quads_per_row);

  float acc = 0.f, acc_x = 0.f;
  float4 xv[kStepUnroll], nx[kStepUnroll];
  VReg vv[kStepUnroll], nv[kStepUnroll];
  int q = q_begin + threadIdx.x;
  if (q_end - q_begin == p.chunk_quads) {
    // full chunk (a multiple of 2 * kStepUnroll * kRowThreads quads): two register sets take
    // turns, no bounds checks and no register copies
    constexpr int kStride = kStepUnroll * kRowThreads;
    const int iters = p.chunk_quads / kStride;          // even
#pragma unroll
    for (int u = 0; u < kStepUnroll; ++u) {
      xv[u] = __ldcs(xin + q + u * kRowThreads);
      load_vel(vel, (size_t)(q + u * kRowThreads), vv[u]);
    }
    for (int it = 0; it < iters; it += 2) {
#pragma unroll
      for (int u = 0; u < kStepUnroll; ++u) {
        nx[u] = __ldcs(xin + q + kStride + u * kRowThreads);
        load_vel(vel, (size_t)(q + kStride + u * kRowThreads), nv[u]);
      }
#pragma unroll
      for (int u = 0; u < kStepUnroll; ++u)
        step_quad<kNoise, kUnitCx, kMean>(p, traj, q + u * kRowThreads, xv[u], vel_f32(vv[u]), xout, acc, acc_x);
      if (it + 2 < iters) {
#pragma unroll
        for (int u = 0; u < kStepUnroll; ++u) {
          xv[u] = __ldcs(xin + q + 2 * kStride + u * kRowThreads);
          load_vel(vel, (size_t)(q + 2 * kStride + u * kRowThreads), vv[u]);
        }
      }
#pragma unroll
      for (int u = 0; u < kStepUnroll; ++u)
        step_quad<kNoise, kUnitCx, kMean>(p, traj, q + kStride + u * kRowThreads, nx[u], vel_f32(nv[u]), xout, acc, acc_x);
      q += 2 * kStride;
    }
    q = q_end;
  } else {
#pragma unroll
    for (int u = 0; u < kStepUnroll; ++u) {
      const int qq = q + u * kRowThreads;
      if (qq < q_end) { xv[u] = __ldcs(xin + qq); load_vel(vel, (size_t)qq, vv[u]); }
    }
  }
  // ragged last chunk of a row: guarded loop
  while (q < q_end) {
    const int nq = q + kStepUnroll * kRowThreads;
#pragma unroll
    for (int u = 0; u < kStepUnroll; ++u) {
      const int qq = nq + u * kRowThreads;
      if (qq < q_end) { nx[u] = __ldcs(xin + qq); load_vel(vel, (size_t)qq, nv[u]); }
    }
#pragma unroll
    for (int u = 0; u < kStepUnroll; ++u) {
      const int qq = q + u * kRowThreads;
      if (qq < q_end) step_quad<kNoise, kUnitCx, kMean>(p, traj, qq, xv[u], vel_f32(vv[u]), xout, acc, acc_x);
    }
#pragma unroll
    for (int u = 0; u < kStepUnroll; ++u) { xv[u] = nx[u]; vv[u] = nv[u]; }
    q = nq;
  }

  if (!kNoise && !kMean) {
    if (chunk == 0 && threadIdx.x == 0) p.logp_out[row] = 0.f;
    return;
  }
  acc = warp_sum(acc * -kTwoLn2);               // sum of squared noise = -2 ln 2 * sum of log2(u1)
  float* logp_out = p.logp_out;
  const double logp_const = p.logp_const, logp_scale = p.logp_scale;
  if (kMean) {
    const float totals[2] = {acc, warp_sum(acc_x)};
    float* xmean_out = p.xmean_out;
    const double inv_d = p.inv_d;
    finish_row_n<2>(totals, row, chunk, p.chunks, p.partials, p.tickets, [=](const double (&sum)[2]) {
      logp_out[row] = kNoise ? (float)((-0.5 * sum[0] - logp_const) * logp_scale) : 0.f;
      xmean_out[row] = (float)(sum[1] * inv_d);
    });
  } else {
    finish_row(acc, row, chunk, p.chunks, p.partials, p.tickets,
               [=](double sum) { logp_out[row] = (float)((-0.5 * sum - logp_const) * logp_scale); });
  }
}

template <typename VelT, bool kMean>
static void dispatch_step(const StepParams& p, bool noise, bool unit_cx, dim3 grid, cudaStream_t st) {
  const dim3 block(kRowThreads);
  if (noise) {
    if (unit_cx) step_kernel<VelT, true, true, kMean><<<grid, block, 0, st>>>(p);
    else         step_kernel<VelT, true, false, kMean><<<grid, block, 0, st>>>(p);
  } else {
    step_kernel<VelT, false, false, kMean><<<grid, block, 0, st>>>(p);
  }
}

int launch_step(int n_rows, int elems, int vel_dtype, const float* x_in, const void* vel,
                const int32_t* src_rows, const int32_t* traj_id, float* x_out, float* logp_out,
                uint64_t seed, int32_t step, double c_x, double c_v, double noise_std,
                int logp_mean, RowScratch scratch, cudaStream_t stream, int rows_in, int32_t* status,
                float* xmean_out) {
  if (n_rows == 0) return PG_OK;
  const RowGeometry geo = row_geometry(n_rows, elems);
  StepParams p;
  p.status = status;
  p.rows_in = rows_in > 0 ? rows_in : n_rows;
  p.x_in = x_in;
  p.vel = vel;
  p.src_rows = src_rows;
  p.traj_id = traj_id;
  p.x_out = x_out;
  p.logp_out = logp_out;
  p.xmean_out = xmean_out;
  p.inv_d = 1.0 / (double)elems;
  p.partials = scratch.partials;
  p.tickets = scratch.tickets;
  p.quads_per_row = elems / 4;
  p.chunk_quads = geo.chunk_quads;
  p.chunks = geo.chunks;
  p.chunk_shift = -1;
  for (int b = 0; b < 31; ++b)
    if (geo.chunks == (1 << b)) p.chunk_shift = b;
  p.step = (uint32_t)step;
  p.c_x = (float)c_x;
  p.c_v = (float)c_v;
  p.neg_scale2 = (float)(-1.3862943611198906 * noise_std * noise_std);
  const double two_pi = 6.283185307179586476925286766559;
  p.logp_const = noise_std > 0.0 ? 0.5 * (double)elems * log(two_pi * noise_std * noise_std) : 0.0;
  p.logp_scale = logp_mean ? 1.0 / (double)elems : 1.0;
  p.rk = make_philox_keys(seed);
  const long long blocks = (long long)n_rows * geo.chunks;
  if (blocks > 0x7FFFFFFFLL) return PG_EINVAL;
  const dim3 grid((unsigned)blocks);
  const bool noise = noise_std > 0.0;
  const bool unit_cx = p.c_x == 1.0f;
  if (vel_dtype == PG_VEL_BF16) {
    if (xmean_out) dispatch_step<__nv_bfloat16, true>(p, noise, unit_cx, grid, stream);
    else           dispatch_step<__nv_bfloat16, false>(p, noise, unit_cx, grid, stream);
  } else {
    if (xmean_out) dispatch_step<float, true>(p, noise, unit_cx, grid, stream);
    else           dispatch_step<float, false>(p, noise, unit_cx, grid, stream);
  }
  PG_LAUNCH_CHECK();
  return PG_OK;
}

// ---------------------------------------------------------------- generator exposure

__global__ void philox_raw_kernel(int64_t n, const uint32_t* ctr, const uint32_t* key,
                                  uint32_t* out) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  PhiloxKeys rk;
  uint32_t a = key[2 * i], b = key[2 * i + 1];
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    rk.k0[r] = a;
    rk.k1[r] = b;
    a += 0x9E3779B9u;
    b += 0xBB67AE85u;
  }
  const uint4 r = philox4x32_10(ctr[4 * i], ctr[4 * i + 1], ctr[4 * i + 2], ctr[4 * i + 3], rk);
  reinterpret_cast<uint4*>(out)[i] = r;
}

int launch_philox_raw(int64_t n, const uint32_t* ctr, const uint32_t* key, uint32_t* out,
                      cudaStream_t stream) {
  if (n == 0) return PG_OK;
  const int64_t blocks = (n + 255) / 256;
  if (blocks > 0x7FFFFFFFLL) return PG_EINVAL;
  philox_raw_kernel<<<(unsigned)blocks, 256, 0, stream>>>(n, ctr, key, out);
  PG_LAUNCH_CHECK();
  return PG_OK;
}

__global__ void normal_rows_kernel(const __grid_constant__ PhiloxKeys rk, uint32_t step,
                                   uint32_t stream_id, int quads_per_row, long long total_quads,
                                   const int32_t* traj_id, float* out) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total_quads) return;
  const int row = (int)(i / quads_per_row);
  const int q = (int)(i - (long long)row * quads_per_row);
  const uint4 r = philox4x32_10((uint32_t)q, step, (uint32_t)traj_id[row], stream_id, rk);
  float4 n;
  normal_pair(r.x, r.y, n.x, n.y);
  normal_pair(r.z, r.w, n.z, n.w);
  reinterpret_cast<float4*>(out)[i] = n;
}

int launch_normal_rows(uint64_t seed, int32_t step, int32_t stream_id, int n_rows, int d,
                       const int32_t* traj_id, float* out, cudaStream_t stream) {
  if (n_rows == 0) return PG_OK;
  const int quads = d / 4;
  const long long total = (long long)n_rows * quads;
  const long long blocks = (total + 255) / 256;
  if (blocks > 0x7FFFFFFFLL) return PG_EINVAL;
  normal_rows_kernel<<<(unsigned)blocks, 256, 0, stream>>>(make_philox_keys(seed), (uint32_t)step,
                                                           (uint32_t)stream_id, quads, total, traj_id, out);
  PG_LAUNCH_CHECK();
  return PG_OK;
}

}  // namespace pg
