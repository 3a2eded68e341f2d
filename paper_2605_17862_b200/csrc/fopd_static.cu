// fopd_token_stats_static: the statistics entry point for callers that must not
// allocate device memory.  Its per-row scratch is a fixed array compiled into
// the library instead of a stream-ordered allocation.
#include <mutex>

#include "host_common.cuh"

using namespace fopd;

// Per-row scratch {lse_s, lse_t, kl, d} for up to FOPD_STATIC_MAX_ROWS rows
// (1 MiB).  Every device that loads the library carries its own copy until the
// process exits.  In host code this name is only a handle for the symbol, not
// a device address: the address is looked up once per device below.
static __device__ __align__(256) float g_static_row_ws[(size_t)FOPD_STATIC_MAX_ROWS * 4];
// Row range of every sample in the chunk, for up to FOPD_STATIC_MAX_SAMPLES samples (256 KiB).
static __device__ __align__(256) unsigned long long g_static_bounds[(size_t)FOPD_STATIC_MAX_SAMPLES * 2];

namespace {

std::mutex g_setup_mutex;
float *g_static_row_ws_addr[kMaxDevices] = {};
unsigned long long *g_static_bounds_addr[kMaxDevices] = {};

// Device address of the scratch array on the current device.  Looked up with
// cudaGetSymbolAddress the first time this device calls in, then cached.
int static_scratch(float **out, unsigned long long **bounds_out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return FOPD_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_static_row_ws_addr[dev]) {
    float *ptr = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void **>(&ptr), g_static_row_ws) != cudaSuccess || !ptr) {
      (void)cudaGetLastError();  // leave no sticky-looking error behind for the caller's next check
      return FOPD_ERR_CUDA;
    }
    unsigned long long *bptr = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void **>(&bptr), g_static_bounds) != cudaSuccess || !bptr) {
      (void)cudaGetLastError();
      return FOPD_ERR_CUDA;
    }
    g_static_row_ws_addr[dev] = ptr;
    g_static_bounds_addr[dev] = bptr;
  }
  *out = g_static_row_ws_addr[dev];
  *bounds_out = g_static_bounds_addr[dev];
  return FOPD_OK;
}

}  // namespace

extern "C" int fopd_token_stats_static(const fopd_chunk *chunk, int32_t B, float *lp_s, float *lp_t,
                                       float *kl, float *ratio, double *acc, int32_t *status,
                                       void *stream) {
  int rc = check_chunk(chunk, B);
  if (rc != FOPD_OK) return rc;
  if (!acc) return FOPD_ERR_NULL;
  if (chunk->n_rows > FOPD_STATIC_MAX_ROWS || B > FOPD_STATIC_MAX_SAMPLES) return FOPD_ERR_SIZE;
  if (chunk->n_rows == 0) return FOPD_OK;
  float *ws = nullptr;
  unsigned long long *bounds = nullptr;
  if ((rc = static_scratch(&ws, &bounds)) != FOPD_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // The sweep writes all four scratch values of every row of the chunk (zeros
  // for rows that are not aligned) before the reduction reads them, and the row
  // ranges of all B samples are reset before they are filled in, so nothing
  // left over from an earlier call is ever read.
  rc = launch_stats(chunk, B, lp_s, lp_t, kl, ratio, ws, status, st);
  if (rc != FOPD_OK) return rc;
  if ((rc = launch_sample_bounds(chunk->sample_id, chunk->n_rows, B, bounds, st)) != FOPD_OK) return rc;
  segment_reduce_kernel<<<B, kSegThreads, 0, st>>>(to_dev(chunk), B, ws, nullptr, 0, bounds_or_null(bounds, B), acc);
  return launch_ok();
}
