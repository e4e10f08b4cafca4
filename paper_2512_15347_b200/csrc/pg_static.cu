// pg_score_static: latent scoring for callers that must not allocate device memory.
//
// Some hosts of this library cannot call cudaMalloc at the point where they need a score: code
// running inside another framework's memory pool whose allocator must see every byte, services
// that pin their device footprint at start-up, or callers sitting in a latency-critical section
// where an allocation (which may synchronise the device) is not acceptable.  pg_score() needs a
// handle, and creating a handle allocates its reduction scratch.  This entry point needs no
// handle: the reduction scratch (per-row partial sums and the per-row arrival counters) lives in
// a fixed array that is part of the library image, so every GPU that loads the library carries
// it (about 300 KB) until the process exits.
//
// The first call on a device looks up the device address of that array; host code cannot use
// the array's name as a pointer (on the host the name denotes a stand-in object, not device
// memory), so the address is obtained with cudaGetSymbolAddress while that device is current.
#include "pg_common.cuh"

#include <mutex>

namespace {

constexpr int kStaticMaxRows = PG_STATIC_MAX_ROWS;
constexpr size_t kStaticMaxPartials = PG_STATIC_MAX_PARTIALS;
constexpr int kMaxDevices = 64;
constexpr int kStaticChunkQuads = 8192;   // 32768 elements per partial sum: the limit the header documents

struct StaticScratch {
  float partials[kStaticMaxPartials];
  unsigned int tickets[kStaticMaxRows];
};

// Scratch of the no-allocation scoring entry point.  Shared by every call on this device.
static __device__ __align__(256) StaticScratch g_score_scratch;

std::mutex g_setup_mutex;
StaticScratch* g_scratch_addr[kMaxDevices] = {};

// Device address of g_score_scratch on the current device (looked up once per device).
int scratch_for_current_device(StaticScratch** out) {
  int dev = 0;
  PG_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return PG_EINVAL;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    PG_CUDA(cudaGetSymbolAddress(&p, g_score_scratch));
    g_scratch_addr[dev] = static_cast<StaticScratch*>(p);
  }
  *out = g_scratch_addr[dev];
  return PG_OK;
}

}  // namespace

extern "C" int pg_score_static(int32_t n_rows, int32_t elems, int32_t vel_dtype,
                               const pg_preview_coef* coef, const float* x, const void* vel,
                               float* scores_out, void* stream) {
  if (n_rows < 0 || elems < 4 || (elems & 3) || !coef) return PG_EINVAL;
  if (vel_dtype != PG_VEL_F32 && vel_dtype != PG_VEL_BF16) return PG_EINVAL;
  if (!(coef->p_x == coef->p_x) || !(coef->p_v == coef->p_v)) return PG_EINVAL;
  if (n_rows == 0) return PG_OK;
  if (!x || !scores_out || (coef->p_v != 0.0 && !vel)) return PG_EINVAL;
  if (((uintptr_t)x & 15) || ((uintptr_t)vel & 15)) return PG_EINVAL;
  // capacity of the built-in scratch: PG_STATIC_MAX_ROWS rows, PG_STATIC_MAX_PARTIALS partial sums
  if (n_rows > kStaticMaxRows) return PG_ECAPACITY;
  const pg::RowGeometry geo = pg::row_geometry(n_rows, elems, kStaticChunkQuads);
  const size_t need = (size_t)n_rows * (size_t)geo.chunks;
  if (need > kStaticMaxPartials) return PG_ECAPACITY;

  StaticScratch* s = nullptr;
  const int rc = scratch_for_current_device(&s);
  if (rc != PG_OK) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  // the array keeps whatever the previous call left: the arrival counters must start at zero
  PG_CUDA(cudaMemsetAsync(s->tickets, 0, (size_t)n_rows * sizeof(unsigned int), st));
  pg::RowScratch scratch{s->partials, s->tickets};
  return pg::launch_score(n_rows, elems, vel_dtype, x, vel, coef->p_x, coef->p_v, scores_out,
                          nullptr, 0, scratch, st, kStaticChunkQuads);
}
