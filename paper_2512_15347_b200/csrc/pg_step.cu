// Fused Euler-Maruyama step + Gaussian policy log-probability (Eq. "euler_method").
//
// One CTA streams one chunk (8192 elements) of one trajectory: x and the prediction are read
// once with 128/64-bit coalesced loads, the noise is generated in registers (one Philox block
// per 4 elements), x' is written once.  The per-trajectory sum of xi^2 is reduced
// thread -> warp (shuffle) -> CTA (shared memory) -> trajectory (fixed-slot partials, finished
// by the last CTA of the row through a wait-free ticket), so the result does not depend on
// the order in which CTAs run.
#include "pg_common.cuh"

namespace pg {

struct StepParams {
  const float* x_in;
  const void* vel;
  const int32_t* src_rows;
  const int32_t* traj_id;
  float* x_out;
  float* logp_out;
  float* partials;
  unsigned int* tickets;
  int quads_per_row;      // d / 4
  int chunks;             // CTAs per row
  uint32_t step;
  float c_x, c_v, noise_std;
  double logp_const;      // d/2 * ln(2 pi noise_std^2)
  double logp_scale;      // 1 or 1/d
  PhiloxKeys rk;
};

__device__ __forceinline__ float4 load_vel4(const float* v, size_t quad) {
  return __ldcs(reinterpret_cast<const float4*>(v) + quad);
}
__device__ __forceinline__ float4 load_vel4(const __nv_bfloat16* v, size_t quad) {
  const uint2 w = __ldcs(reinterpret_cast<const uint2*>(v) + quad);
  float4 r;
  r.x = __uint_as_float(w.x << 16);
  r.y = __uint_as_float(w.x & 0xFFFF0000u);
  r.z = __uint_as_float(w.y << 16);
  r.w = __uint_as_float(w.y & 0xFFFF0000u);
  return r;
}

template <typename VelT, bool kNoise>
__global__ void __launch_bounds__(kRowThreads)
step_kernel(const __grid_constant__ StepParams p) {
  const int row = blockIdx.x / p.chunks;
  const int chunk = blockIdx.x - row * p.chunks;
  const int src = p.src_rows ? p.src_rows[row] : row;
  const uint32_t traj = (uint32_t)p.traj_id[row];

  const size_t in_base = (size_t)src * p.quads_per_row;
  const size_t out_base = (size_t)row * p.quads_per_row;
  const VelT* vel = reinterpret_cast<const VelT*>(p.vel);
  const int q0 = chunk * kChunkQuads + threadIdx.x;

  float acc = 0.f;
#pragma unroll
  for (int half = 0; half < 2; ++half) {
    constexpr int kU = kQuadsPerThread / 2;
    float4 xv[kU], vv[kU];
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      const int q = q0 + (half * kU + u) * kRowThreads;
      if (q < p.quads_per_row) {
        xv[u] = __ldcs(reinterpret_cast<const float4*>(p.x_in) + in_base + q);
        vv[u] = load_vel4(vel, in_base + q);
      }
    }
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      const int q = q0 + (half * kU + u) * kRowThreads;
      if (q < p.quads_per_row) {
        float4 m;
        m.x = fmaf(p.c_v, vv[u].x, p.c_x * xv[u].x);
        m.y = fmaf(p.c_v, vv[u].y, p.c_x * xv[u].y);
        m.z = fmaf(p.c_v, vv[u].z, p.c_x * xv[u].z);
        m.w = fmaf(p.c_v, vv[u].w, p.c_x * xv[u].w);
        if (kNoise) {
          const uint4 r = philox4x32_10((uint32_t)q, p.step, traj, 0u, p.rk);
          float n0, n1, n2, n3;
          normal_pair(r.x, r.y, n0, n1);
          normal_pair(r.z, r.w, n2, n3);
          acc += (n0 * n0 + n1 * n1) + (n2 * n2 + n3 * n3);
          m.x = fmaf(p.noise_std, n0, m.x);
          m.y = fmaf(p.noise_std, n1, m.y);
          m.z = fmaf(p.noise_std, n2, m.z);
          m.w = fmaf(p.noise_std, n3, m.w);
        }
        __stcs(reinterpret_cast<float4*>(p.x_out) + out_base + q, m);
      }
    }
  }

  if (!kNoise) {
    if (chunk == 0 && threadIdx.x == 0) p.logp_out[row] = 0.f;
    return;
  }

  // CTA reduction in a fixed shape
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
        p.logp_out[row] = (float)((-0.5 * (double)v - p.logp_const) * p.logp_scale);
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
  // last CTA of this row: all partials are visible; add them in slot order
  if (threadIdx.x < 32) {
    __threadfence();
    double s = 0.0;
    for (int c = threadIdx.x; c < p.chunks; c += 32)
      s += (double)__ldcg(&p.partials[(size_t)row * p.chunks + c]);
    s = warp_sum(s);
    if (threadIdx.x == 0) {
      p.logp_out[row] = (float)((-0.5 * s - p.logp_const) * p.logp_scale);
      p.tickets[row] = 0u;   // ready for the next launch
    }
  }
}

int launch_step(int n_rows, int elems, int vel_dtype, const float* x_in, const void* vel,
                const int32_t* src_rows, const int32_t* traj_id, float* x_out, float* logp_out,
                uint64_t seed, int32_t step, double c_x, double c_v, double noise_std,
                int logp_mean, RowScratch scratch, cudaStream_t stream) {
  if (n_rows == 0) return PG_OK;
  StepParams p;
  p.x_in = x_in;
  p.vel = vel;
  p.src_rows = src_rows;
  p.traj_id = traj_id;
  p.x_out = x_out;
  p.logp_out = logp_out;
  p.partials = scratch.partials;
  p.tickets = scratch.tickets;
  p.quads_per_row = elems / 4;
  p.chunks = chunks_per_row(elems);
  p.step = (uint32_t)step;
  p.c_x = (float)c_x;
  p.c_v = (float)c_v;
  p.noise_std = (float)noise_std;
  const double two_pi = 6.283185307179586476925286766559;
  // the device scales the noise by the fp32 value of noise_std; the density uses the same
  const double ns = (double)p.noise_std;
  p.logp_const = noise_std > 0.0 ? 0.5 * (double)elems * log(two_pi * ns * ns) : 0.0;
  p.logp_scale = logp_mean ? 1.0 / (double)elems : 1.0;
  p.rk = make_philox_keys(seed);
  const long long blocks = (long long)n_rows * p.chunks;
  if (blocks > 0x7FFFFFFFLL) return PG_EINVAL;
  const dim3 grid((unsigned)blocks), block(kRowThreads);
  const bool noise = noise_std > 0.0;
  if (vel_dtype == PG_VEL_BF16) {
    if (noise) step_kernel<__nv_bfloat16, true><<<grid, block, 0, stream>>>(p);
    else       step_kernel<__nv_bfloat16, false><<<grid, block, 0, stream>>>(p);
  } else {
    if (noise) step_kernel<float, true><<<grid, block, 0, stream>>>(p);
    else       step_kernel<float, false><<<grid, block, 0, stream>>>(p);
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
                                   uint32_t stream_id, int quads_per_row, const int32_t* traj_id,
                                   float* out) {
  const int row = blockIdx.y;
  const int q = blockIdx.x * blockDim.x + threadIdx.x;
  if (q >= quads_per_row) return;
  const uint4 r = philox4x32_10((uint32_t)q, step, (uint32_t)traj_id[row], stream_id, rk);
  float4 n;
  normal_pair(r.x, r.y, n.x, n.y);
  normal_pair(r.z, r.w, n.z, n.w);
  reinterpret_cast<float4*>(out)[(size_t)row * quads_per_row + q] = n;
}

int launch_normal_rows(uint64_t seed, int32_t step, int32_t stream_id, int n_rows, int d,
                       const int32_t* traj_id, float* out, cudaStream_t stream) {
  if (n_rows == 0) return PG_OK;
  if (n_rows > 65535) return PG_EINVAL;
  const int quads = d / 4;
  const dim3 grid((quads + 255) / 256, n_rows);
  normal_rows_kernel<<<grid, 256, 0, stream>>>(make_philox_keys(seed), (uint32_t)step,
                                               (uint32_t)stream_id, quads, traj_id, out);
  PG_LAUNCH_CHECK();
  return PG_OK;
}

}  // namespace pg
