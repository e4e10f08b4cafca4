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

}  // namespace pg
