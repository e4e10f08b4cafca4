// Survivor compaction of row arrays (Section 5.1: early-terminated trajectories take no further
// steps): dst row g*k + p = src row g*n_prev + keep_idx[g*k + p].  Pure gather; each CTA moves
// one 32 KB piece of one row with the widest access the row alignment allows.
#include "pg_common.cuh"

namespace pg {

constexpr int kCompactThreads = 256;
constexpr size_t kCompactPiece = 32768;   // bytes per CTA

__device__ __forceinline__ uint4 ldcs_word(const uint4* p) { return __ldcs(p); }
__device__ __forceinline__ void stcs_word(uint4* p, const uint4& v) { __stcs(p, v); }
template <typename T> __device__ __forceinline__ T ldcs_word(const T* p) { return *p; }
template <typename T> __device__ __forceinline__ void stcs_word(T* p, const T& v) { *p = v; }

template <typename T>
__global__ void __launch_bounds__(kCompactThreads)
compact_kernel(const int32_t* keep_idx, const unsigned char* src, unsigned char* dst,
               size_t row_bytes, int n_prev, int k, int pieces, int32_t* status) {
  const int row = blockIdx.x / pieces;
  const int piece = blockIdx.x - row * pieces;
  const int g = row / k;
  const int slot = keep_idx[row];
  if ((unsigned int)slot >= (unsigned int)n_prev) {       // never dereference a bad slot
    if (threadIdx.x == 0 && piece == 0 && status) atomicOr(status, 4);
    return;
  }
  const size_t begin = (size_t)piece * kCompactPiece;
  const size_t end = (begin + kCompactPiece < row_bytes) ? begin + kCompactPiece : row_bytes;
  const T* s = reinterpret_cast<const T*>(src + ((size_t)g * n_prev + slot) * row_bytes + begin);
  T* d = reinterpret_cast<T*>(dst + (size_t)row * row_bytes + begin);
  const size_t count = (end - begin) / sizeof(T);
  constexpr size_t kFull = kCompactPiece / sizeof(T);
  constexpr int kPerThread = (int)(kFull / kCompactThreads);
  if constexpr (sizeof(T) == 16) if (count == kFull) {
    // full piece of 16-byte words: all loads of the thread in flight before the first store,
    // streaming hints on both sides (every byte is touched once)
    T r[kPerThread];
#pragma unroll
    for (int u = 0; u < kPerThread; ++u) r[u] = ldcs_word(s + threadIdx.x + u * kCompactThreads);
#pragma unroll
    for (int u = 0; u < kPerThread; ++u) stcs_word(d + threadIdx.x + u * kCompactThreads, r[u]);
    return;
  }
  for (size_t i = threadIdx.x; i < count; i += kCompactThreads) d[i] = s[i];
}

// Narrow rows (a few bytes, e.g. one fp32 per trajectory): one thread per row.
template <typename T>
__global__ void compact_small_kernel(const int32_t* keep_idx, const T* src, T* dst, int n_rows,
                                     int n_prev, int k, int per_row, int32_t* status) {
  const int row = blockIdx.x * blockDim.x + threadIdx.x;
  if (row >= n_rows) return;
  const int g = row / k;
  if ((unsigned int)keep_idx[row] >= (unsigned int)n_prev) {
    if (status) atomicOr(status, 4);
    return;
  }
  const size_t s = ((size_t)g * n_prev + keep_idx[row]) * per_row;
  for (int i = 0; i < per_row; ++i) dst[(size_t)row * per_row + i] = src[s + i];
}

int launch_compact(int n_groups, int n_prev, int k, const int32_t* keep_idx, const void* src,
                   void* dst, size_t row_bytes, cudaStream_t stream, int32_t* status) {
  const long long rows = (long long)n_groups * k;
  if (rows == 0) return PG_OK;
  const uintptr_t a = (uintptr_t)src | (uintptr_t)dst | (uintptr_t)row_bytes;
  if (row_bytes <= 64) {
    const unsigned blocks = (unsigned)((rows + 255) / 256);
    if ((a & 3) == 0)
      compact_small_kernel<uint32_t><<<blocks, 256, 0, stream>>>(
          keep_idx, (const uint32_t*)src, (uint32_t*)dst, (int)rows, n_prev, k, (int)(row_bytes / 4), status);
    else
      compact_small_kernel<unsigned char><<<blocks, 256, 0, stream>>>(
          keep_idx, (const unsigned char*)src, (unsigned char*)dst, (int)rows, n_prev, k, (int)row_bytes, status);
    PG_LAUNCH_CHECK();
    return PG_OK;
  }
  const int pieces = (int)((row_bytes + kCompactPiece - 1) / kCompactPiece);
  const long long blocks = rows * pieces;
  if (blocks > 0x7FFFFFFFLL) return PG_EINVAL;
  const unsigned char* s = (const unsigned char*)src;
  unsigned char* d = (unsigned char*)dst;
  if ((a & 15) == 0)
    compact_kernel<uint4><<<(unsigned)blocks, kCompactThreads, 0, stream>>>(keep_idx, s, d, row_bytes, n_prev, k, pieces, status);
  else if ((a & 3) == 0)
    compact_kernel<uint32_t><<<(unsigned)blocks, kCompactThreads, 0, stream>>>(keep_idx, s, d, row_bytes, n_prev, k, pieces, status);
  else
    compact_kernel<unsigned char><<<(unsigned)blocks, kCompactThreads, 0, stream>>>(keep_idx, s, d, row_bytes, n_prev, k, pieces, status);
  PG_LAUNCH_CHECK();
  return PG_OK;
}

// ---------------------------------------------------------------- survivors' history

// Row of every final survivor at every step.  One thread per final survivor walks the stages
// from the last to the first: behind stage i its slot is `slot`, in front of it the slot is
// keep_idx_i[g * k_i + slot].  Steps from stage_step[i] on (up to the next stage) use the slot
// behind stage i; steps before the first stage use the original slot.
struct SurvivorParams {
  const int32_t* keep_idx;      // packed stage after stage: [G * k_0], [G * k_1], ...
  int32_t* rows_out;            // [T, G * K]
  int32_t* status;              // bit 2: a kept slot outside its group
  int n_groups, n_expand, n_steps, n_stages, k_final;
  int stage_step[PG_MAX_STAGES];
  int stage_keep[PG_MAX_STAGES];
  long long stage_off[PG_MAX_STAGES];   // offset of stage i in keep_idx
};

__global__ void __launch_bounds__(256) survivor_rows_kernel(const __grid_constant__ SurvivorParams p) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  const int n_final = p.n_groups * p.k_final;
  if (j >= n_final) return;
  const int g = j / p.k_final;
  int slot = j - g * p.k_final;
  int t_hi = p.n_steps;                                   // steps [t_lo, t_hi) use the current slot
  for (int i = p.n_stages - 1; i >= -1; --i) {
    const int t_lo = i >= 0 ? p.stage_step[i] : 0;
    const int k_here = i >= 0 ? p.stage_keep[i] : p.n_expand;
    for (int t = t_lo; t < t_hi; ++t) p.rows_out[(size_t)t * n_final + j] = g * k_here + slot;
    if (i < 0) break;
    const int k_before = i > 0 ? p.stage_keep[i - 1] : p.n_expand;
    const int prev = p.keep_idx[p.stage_off[i] + (long long)g * k_here + slot];
    if ((unsigned int)prev >= (unsigned int)k_before) {   // never used as an index
      if (p.status) atomicOr(p.status, 4);
      slot = 0;
    } else {
      slot = prev;
    }
    t_hi = t_lo;
  }
}

int launch_survivor_rows(int n_groups, int n_expand, int n_steps, int n_stages, const int32_t* stage_step,
                         const int32_t* stage_keep, const int32_t* keep_idx, int32_t* rows_out,
                         int32_t* status, cudaStream_t stream) {
  if (n_stages > PG_MAX_STAGES) return PG_ECAPACITY;
  SurvivorParams p;
  p.keep_idx = keep_idx;
  p.rows_out = rows_out;
  p.status = status;
  p.n_groups = n_groups;
  p.n_expand = n_expand;
  p.n_steps = n_steps;
  p.n_stages = n_stages;
  long long off = 0;
  for (int i = 0; i < n_stages; ++i) {
    p.stage_step[i] = stage_step[i];
    p.stage_keep[i] = stage_keep[i];
    p.stage_off[i] = off;
    off += (long long)n_groups * stage_keep[i];
  }
  p.k_final = n_stages > 0 ? stage_keep[n_stages - 1] : n_expand;
  const long long n_final = (long long)n_groups * p.k_final;
  if (n_final == 0 || n_steps == 0) return PG_OK;
  survivor_rows_kernel<<<(unsigned)((n_final + 255) / 256), 256, 0, stream>>>(p);
  PG_LAUNCH_CHECK();
  return PG_OK;
}

// logp_out[t][j] = logp_packed[offset of step t + rows[t][j]]: the survivors' log-prob history
// out of the per-step arrays packed step after step.
__global__ void __launch_bounds__(256)
survivor_logp_kernel(const int32_t* __restrict__ rows, const float* __restrict__ logp_packed,
                     float* __restrict__ logp_out, const long long* __restrict__ step_off,
                     int n_steps, int n_final, int32_t* status) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (long long)n_steps * n_final) return;
  const int t = (int)(i / n_final);
  const long long lo = step_off[t], hi = step_off[t + 1];
  const long long r = rows[i];
  if (r < 0 || lo + r >= hi) {
    if (status) atomicOr(status, 4);
    return;
  }
  logp_out[i] = logp_packed[lo + r];
}

int launch_survivor_logp(const int32_t* rows, const float* logp_packed, float* logp_out,
                         const long long* step_off_dev, int n_steps, int n_final, int32_t* status,
                         cudaStream_t stream) {
  const long long total = (long long)n_steps * n_final;
  if (total == 0) return PG_OK;
  survivor_logp_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(rows, logp_packed, logp_out,
                                                                           step_off_dev, n_steps, n_final, status);
  PG_LAUNCH_CHECK();
  return PG_OK;
}

}  // namespace pg
