// Host-side helpers shared by the entry points of libfopd: argument checks,
// the memory pool for temporaries and the launch of the statistics sweep.
#pragma once

#include <cmath>
#include <mutex>

#include "stream_kernels.cuh"

namespace fopd {

static inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static inline int check_chunk(const fopd_chunk *c, int32_t B, bool needs_teacher = true) {
  if (!c) return FOPD_ERR_NULL;
  if (c->dtype != FOPD_BF16 && c->dtype != FOPD_F32) return FOPD_ERR_DTYPE;
  if (c->loss_kind != FOPD_LOSS_FULL_KL && c->loss_kind != FOPD_LOSS_SAMPLED_KL) return FOPD_ERR_KIND;
  if (c->n_rows < 0 || c->vocab <= 0 || c->row_stride < c->vocab || B <= 0) return FOPD_ERR_SIZE;
  if (c->vocab > (int64_t)1 << 30 || c->n_rows > (int64_t)1 << 40) return FOPD_ERR_SIZE;
  if (c->n_rows == 0) return FOPD_OK;
  if (!c->student || (needs_teacher && !c->teacher) || !c->behav_logprob || !c->tokens || !c->mask || !c->sample_id)
    return FOPD_ERR_NULL;
  const int64_t esz = c->dtype == FOPD_BF16 ? 2 : 4;
  if (!aligned16(c->student) || (needs_teacher && !aligned16(c->teacher)) || (c->row_stride * esz) % 16 != 0)
    return FOPD_ERR_ALIGN;
  return FOPD_OK;
}

static inline ChunkDev to_dev(const fopd_chunk *c) {
  ChunkDev d;
  d.student = c->student;
  d.teacher = c->teacher;
  d.behav = c->behav_logprob;
  d.tokens = c->tokens;
  d.mask = c->mask;
  d.sid = c->sample_id;
  d.n_rows = c->n_rows;
  d.vocab = c->vocab;
  d.stride = c->row_stride;
  d.kind = c->loss_kind;
  return d;
}

static inline int check_params(const fopd_params &p) {
  if (!std::isfinite(p.alpha) || !std::isfinite(p.beta) || !std::isfinite(p.xi) || !std::isfinite(p.lambda))
    return FOPD_ERR_PARAM;
  if (p.alpha < 0.f || p.beta < 0.f) return FOPD_ERR_PARAM;
  return FOPD_OK;
}

static inline int launch_ok() { return cudaGetLastError() == cudaSuccess ? FOPD_OK : FOPD_ERR_CUDA; }

// Stream-ordered temporaries come from a memory pool of the library's own (one per device)
// that keeps what it has been given: with the device's default pool a synchronisation
// between two calls hands the memory back to the driver and the next call pays for a
// fresh allocation, which costs more than the kernels.
constexpr int kMaxDevices = 64;
struct ScratchPools {
  std::mutex mu;
  cudaMemPool_t pools[kMaxDevices] = {};
};
inline ScratchPools &scratch_pools() {
  static ScratchPools p;  // one per process (inline function: one instance across translation units)
  return p;
}

static inline int scratch_alloc(void **ptr, size_t bytes, cudaStream_t st) {
  ScratchPools &sp = scratch_pools();
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return FOPD_ERR_CUDA;
  cudaMemPool_t pool;
  {
    std::lock_guard<std::mutex> lock(sp.mu);
    if (!sp.pools[dev]) {
      cudaMemPoolProps props = {};
      props.allocType = cudaMemAllocationTypePinned;
      props.location.type = cudaMemLocationTypeDevice;
      props.location.id = dev;
      cudaMemPool_t created;
      if (cudaMemPoolCreate(&created, &props) != cudaSuccess) return FOPD_ERR_CUDA;
      unsigned long long keep = ~0ull;
      if (cudaMemPoolSetAttribute(created, cudaMemPoolAttrReleaseThreshold, &keep) != cudaSuccess) {
        (void)cudaMemPoolDestroy(created);
        return FOPD_ERR_CUDA;
      }
      sp.pools[dev] = created;
    }
    pool = sp.pools[dev];
  }
  return cudaMallocFromPoolAsync(ptr, bytes, pool, st) == cudaSuccess ? FOPD_OK : FOPD_ERR_CUDA;
}

// Gives the memory the current device's pool holds but no pending call uses back to the driver.
static inline int scratch_release() {
  ScratchPools &sp = scratch_pools();
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return FOPD_ERR_CUDA;
  std::lock_guard<std::mutex> lock(sp.mu);
  if (!sp.pools[dev]) return FOPD_OK;
  return cudaMemPoolTrimTo(sp.pools[dev], 0) == cudaSuccess ? FOPD_OK : FOPD_ERR_CUDA;
}

// Enqueues the pass that finds every sample's row range in a chunk (bounds: [B, 2] 64-bit).
static inline int launch_sample_bounds(const int32_t *sid, int64_t n_rows, int32_t B, unsigned long long *bounds,
                                       cudaStream_t st) {
  if (B <= kFewSamples) return FOPD_OK;  // the reductions find the ranges themselves (see bounds_or_null)
  sample_bounds_init_kernel<<<(unsigned)((B + 255) / 256), 256, 0, st>>>(B, bounds);
  if (n_rows > 0) sample_bounds_kernel<<<(unsigned)((n_rows + 255) / 256), 256, 0, st>>>(sid, n_rows, B, bounds);
  return launch_ok();
}
static inline size_t bounds_bytes(int32_t B) { return (size_t)B * 2 * sizeof(unsigned long long); }
// What the reduction kernels are handed: the ranges launch_sample_bounds filled in, or NULL for a
// batch of few samples, whose reduction blocks scan the ids themselves.
static inline const unsigned long long *bounds_or_null(const unsigned long long *bounds, int32_t B) {
  return B <= kFewSamples ? nullptr : bounds;
}

// The per-sample reduction of a chunk's row statistics with its row ranges in a temporary of
// the library's pool.  mode 0: acc[B,4] +=; mode 1: loss_acc[B,2] += (see segment_reduce_kernel).
static inline int launch_segment_reduce(const ChunkDev &d, int32_t B, const float *row_ws, const float *coef, int mode,
                                        double *out, cudaStream_t st) {
  unsigned long long *bounds = nullptr;
  int rc = scratch_alloc(reinterpret_cast<void **>(&bounds), bounds_bytes(B), st);
  if (rc != FOPD_OK) return rc;
  rc = launch_sample_bounds(d.sid, d.n_rows, B, bounds, st);
  if (rc == FOPD_OK) {
    segment_reduce_kernel<<<B, kSegThreads, 0, st>>>(d, B, row_ws, coef, mode, bounds_or_null(bounds, B), out);
    rc = launch_ok();
  }
  if (cudaFreeAsync(bounds, st) != cudaSuccess) rc = FOPD_ERR_CUDA;
  return rc;
}

// One CTA per row.
static inline unsigned row_grid(int64_t n_rows) { return (unsigned)(n_rows < kMaxGrid ? n_rows : kMaxGrid); }

// Enqueues the statistics sweep of a chunk into row_ws (and the optional
// per-row outputs).
static inline int launch_stats(const fopd_chunk *c, int32_t B, float *lp_s, float *lp_t, float *kl, float *ratio,
                 float *row_ws, int32_t *status, cudaStream_t st) {
  const ChunkDev d = to_dev(c);
  const unsigned grid = row_grid(c->n_rows);
  const bool short_row = c->vocab / (c->dtype == FOPD_BF16 ? 8 : 4) < kShortRowVecs;
#define FOPD_LAUNCH_STATS(DT, T) \
  token_stats_kernel<DT, T><<<grid, T, 0, st>>>(d, B, lp_s, lp_t, kl, ratio, row_ws, status)
  if (c->dtype == FOPD_BF16) {
    if (short_row) FOPD_LAUNCH_STATS(FOPD_BF16, kStatsThreadsShortRow);
    else FOPD_LAUNCH_STATS(FOPD_BF16, kStatsThreads);
  } else {
    if (short_row) FOPD_LAUNCH_STATS(FOPD_F32, kStatsThreadsShortRow);
    else FOPD_LAUNCH_STATS(FOPD_F32, kStatsThreads);
  }
#undef FOPD_LAUNCH_STATS
  return launch_ok();
}


}  // namespace fopd
