// C ABI of libfopd: argument checks on the host, kernel launches on the
// caller's stream.  See include/fopd.h for the contract of every entry point.
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <mutex>
#include <vector>

#include "cluster_kernel.cuh"
#include "host_common.cuh"

using namespace fopd;

namespace fopd {
int host_step_release();  // fopd_host.cu: the host-buffer step's streams and events on the current device
}

namespace {

// Planning and launching both set per-function attributes of the on-chip kernel: one lock for both.
std::mutex g_fused_mu;

constexpr int kNotApplicable = 1;  // the on-chip kernel cannot take this shape; use the streaming pair

// Launch shape of the on-chip kernel for one (device, dtype, vocabulary): cluster size, compute
// warps, vectors per compute thread, shared memory and how many clusters are resident.
struct FusedPlan {
  int cluster = 0;        // 0: no shape fits (or the streaming pair is faster), use the streaming pair
  int nv = 0, warps = 0;  // template parameters: vectors of a slice per compute thread, compute warps
  int slice_vecs = 0;
  size_t smem = 0;
  int max_clusters = 0;
};

template <int DT>
const void *fused_kernel_for(int nv, int warps) {
#define X(N, W) \
  if (nv == N && warps == W) return reinterpret_cast<const void *>(&fused_cluster_kernel<DT, N, W>);
  FOPD_FUSED_SHAPES(X)
#undef X
  return nullptr;
}

// The instantiated (vectors per thread, compute warps) pair that covers a slice of `slice`
// vectors with the fewest slots (slots beyond the slice are worked on all the same); among
// equals the one with more warps.  false: the slice is too long for any.
static bool fused_shape_for(int64_t slice, int *nv, int *warps) {
  int64_t best = -1;
#define X(N, W)                                                                                       \
  if ((int64_t)N * W * 32 >= slice && (best < 0 || (int64_t)N * W < best || ((int64_t)N * W == best && W > *warps))) { \
    best = (int64_t)N * W;                                                                             \
    *nv = N;                                                                                           \
    *warps = W;                                                                                        \
  }
  FOPD_FUSED_SHAPES(X)
#undef X
  return best >= 0;
}

static int set_fused_attributes(const void *kernel, int C, size_t smem) {
  // (all of the SM's configurable memory as shared memory: the kernel hardly uses the L1, and the
  // small CTAs that write the zero rows beside it need room for their buffers)
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess ||
      cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, C > 8 ? 1 : 0) != cudaSuccess) {
    (void)cudaGetLastError();
    return FOPD_ERR_CUDA;
  }
  return FOPD_OK;
}

static void fused_launch_config(cudaLaunchConfig_t *cfg, cudaLaunchAttribute *attr, int C, int warps, size_t smem,
                                unsigned grid, cudaStream_t st) {
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = C;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  *cfg = cudaLaunchConfig_t{};
  cfg->blockDim = dim3(warps * 32 + 32);
  cfg->gridDim = dim3(grid);
  cfg->dynamicSmemBytes = smem;
  cfg->stream = st;
  cfg->attrs = attr;
  cfg->numAttrs = 1;
}

// Shape for one cluster size, or plan->cluster = 0 if that size cannot hold the row: a CTA's
// slice must be within what its compute threads take (kFusedMaxNV vectors each) and two student
// and three teacher slices must fit its shared memory.
template <int DT>
int fused_plan_for_cluster(int64_t nvec, int C, int max_optin, FusedPlan *plan) {
  *plan = FusedPlan();
  const size_t fixed = ((sizeof(ClusterShared) + 127) & ~size_t(127));
  const int64_t slice = (nvec + C - 1) / C;
  int nv = 0, warps = 0;
  const size_t smem = fixed + (size_t)kSliceBufs * (size_t)slice * 16;
  // (one copy barrier counts < 2^20 bytes)
  if (!fused_shape_for(slice, &nv, &warps) || smem > (size_t)max_optin || slice * 16 >= (1 << 20)) return FOPD_OK;
  const void *kernel = fused_kernel_for<DT>(nv, warps);
  int rc = set_fused_attributes(kernel, C, smem);
  if (rc != FOPD_OK) return rc;
  cudaLaunchConfig_t cfg;
  cudaLaunchAttribute attr[1];
  fused_launch_config(&cfg, attr, C, warps, smem, (unsigned)C, nullptr);
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, kernel, &cfg) != cudaSuccess) {
    (void)cudaGetLastError();
    n = 0;
  }
  if (n < 1) return FOPD_OK;
  plan->cluster = C;
  plan->nv = nv;
  plan->warps = warps;
  plan->slice_vecs = (int)slice;
  plan->smem = smem;
  plan->max_clusters = n;
  return FOPD_OK;
}

// Picks the cluster size that keeps the most CTAs resident (how many clusters of a given size
// fit depends on how the SMs are grouped); among equals the smaller cluster (a shorter
// exchange).  pin > 0: that cluster size or nothing; pin < 0: the streaming pair.
template <int DT>
int make_fused_plan(int64_t nvec, int pin, FusedPlan *plan) {
  *plan = FusedPlan();
  if (pin < 0) return FOPD_OK;
  int dev = 0, max_optin = 0, n_sm = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&max_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n_sm < 1)
    return FOPD_ERR_CUDA;
  FusedPlan best;
  for (int C = 1; C <= kMaxClusterSize; ++C) {
    if (pin > 0 && pin != C) continue;
    FusedPlan cand;
    int rc = fused_plan_for_cluster<DT>(nvec, C, max_optin, &cand);
    if (rc != FOPD_OK) return rc;
    if (cand.cluster && cand.max_clusters * cand.cluster > best.max_clusters * best.cluster) best = cand;
  }
  // The on-chip kernel is bound by instruction issue, so its rate follows the number of resident
  // CTAs; the two streaming sweeps move five thirds of the bytes at the memory system's rate.
  // With fewer than about two thirds of the SMs busy (very long rows) the streaming pair wins.
  if (pin == 0 && best.cluster && best.max_clusters * best.cluster * 3 < n_sm * 2) best = FusedPlan();
  *plan = best;
  return FOPD_OK;
}

struct PlanEntry {
  int dev, dtype;
  int64_t nvec;
  int pin;      // 0 automatic, > 0 cluster size set by the caller, < 0 streaming pair set by the caller
  bool planned;
  FusedPlan plan;
};
std::vector<PlanEntry> g_plans;  // guarded by g_fused_mu

// Entry of (current device, dtype, nvec), created on first use.  Caller holds g_fused_mu.
PlanEntry *plan_entry(int dtype, int64_t nvec) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return nullptr;
  for (PlanEntry &e : g_plans)
    if (e.dev == dev && e.dtype == dtype && e.nvec == nvec) return &e;
  g_plans.push_back({dev, dtype, nvec, 0, false, FusedPlan()});
  return &g_plans.back();
}

template <int DT>
int fused_plan(int64_t nvec, FusedPlan *plan) {
  std::lock_guard<std::mutex> lock(g_fused_mu);
  PlanEntry *e = plan_entry(DT, nvec);
  if (!e) return FOPD_ERR_CUDA;
  if (!e->planned) {
    int rc = make_fused_plan<DT>(nvec, e->pin, &e->plan);
    if (rc != FOPD_OK) return rc;
    e->planned = true;
  }
  *plan = e->plan;
  return FOPD_OK;
}

// Fused on-chip forward + backward (cluster_kernel.cuh).  tmp holds [n_rows, 4] row
// statistics (out) followed by [n_rows] row weights (scratch).
template <int DT>
int launch_fused(const fopd_chunk *chunk, int32_t B, const float *coef, float lambda, void *dlogits,
                 float *tmp, int32_t *status, cudaStream_t st) {
  using E = Elem<DT>;
  const int64_t nvec = chunk->vocab / E::kPerVec;
  if (nvec < 1) return kNotApplicable;
  FusedPlan plan;
  int rc = fused_plan<DT>(nvec, &plan);
  if (rc != FOPD_OK) return rc;
  if (!plan.cluster || plan.max_clusters < 1) return kNotApplicable;
  const int C = plan.cluster;
  const void *kernel = fused_kernel_for<DT>(plan.nv, plan.warps);
  float *row_cf = tmp + 4 * chunk->n_rows;
  const ChunkDev d = to_dev(chunk);
  row_weight_kernel<<<(unsigned)((chunk->n_rows + 255) / 256), 256, 0, st>>>(d, B, coef, status, row_cf);
  if ((rc = launch_ok()) != FOPD_OK) return rc;
  const int64_t clusters = chunk->n_rows < plan.max_clusters ? chunk->n_rows : plan.max_clusters;
  cudaLaunchConfig_t cfg;
  cudaLaunchAttribute attr[1];
  fused_launch_config(&cfg, attr, C, plan.warps, plan.smem, (unsigned)(clusters * C), st);
  FusedArgs a;
  a.c = d;
  a.lambda = lambda;
  a.dlogits = dlogits;
  a.row_cf = row_cf;
  a.row_ws = tmp;
  a.status = status;
  a.slice_vecs = plan.slice_vecs;
  a.wait_cycles = kWaitCycles;
  void *args[] = {&a};
  // the attributes are per function, and the plan of another vocabulary may have changed them:
  // set them and launch under one lock, so that a call from another thread cannot come between
  {
    std::lock_guard<std::mutex> lock(g_fused_mu);
    if ((rc = set_fused_attributes(kernel, C, plan.smem)) != FOPD_OK) return rc;
    if (cudaLaunchKernelExC(&cfg, kernel, args) != cudaSuccess) {
      (void)cudaGetLastError();
      return FOPD_ERR_CUDA;
    }
  }
  // the zeros of the rows that are not differentiated, beside the on-chip kernel (see zero_rows_kernel)
  cudaLaunchAttribute zattr[1];
  zattr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  zattr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t zcfg = cudaLaunchConfig_t{};
  zcfg.blockDim = dim3(32);
  zcfg.gridDim = dim3(row_grid(chunk->n_rows));
  zcfg.dynamicSmemBytes = kZeroBufBytes;
  zcfg.stream = st;
  zcfg.attrs = zattr;
  zcfg.numAttrs = 1;
  const float *row_cf_c = row_cf;
  if (cudaLaunchKernelEx(&zcfg, zero_rows_kernel<DT>, d, row_cf_c, dlogits) != cudaSuccess) {
    (void)cudaGetLastError();
    return FOPD_ERR_CUDA;
  }
  return FOPD_OK;
}

}  // namespace

extern "C" {

int fopd_version(void) { return FOPD_VERSION; }

const char *fopd_strerror(int code) {
  switch (code) {
    case FOPD_OK: return "ok";
    case FOPD_ERR_NULL: return "a required pointer is NULL";
    case FOPD_ERR_ALIGN: return "logits base, row pitch or workspace not 16-byte aligned";
    case FOPD_ERR_SIZE: return "bad size (negative, row_stride < vocab, or too large)";
    case FOPD_ERR_DTYPE: return "dtype must be FOPD_BF16 or FOPD_F32";
    case FOPD_ERR_PARAM: return "alpha/beta must be >= 0 and all parameters finite";
    case FOPD_ERR_CUDA: return "a CUDA runtime call failed";
    case FOPD_ERR_ALIAS: return "dlogits overlaps student or teacher";
    case FOPD_ERR_DEVICE: return "device status word is non-zero (bad token/sample id, staleness, length or timeout)";
    case FOPD_ERR_KIND: return "loss_kind unknown or not supported by this entry point";
    default: return "unknown fopd status";
  }
}

int fopd_token_stats(const fopd_chunk *chunk, int32_t B, float *lp_s, float *lp_t, float *kl,
                     float *ratio, float *row_ws, double *acc, int32_t *status, void *stream) {
  int rc = check_chunk(chunk, B);
  if (rc != FOPD_OK) return rc;
  if (!acc) return FOPD_ERR_NULL;
  if (row_ws && !aligned16(row_ws)) return FOPD_ERR_ALIGN;
  if (chunk->n_rows == 0) return FOPD_OK;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // one temporary: the samples' row ranges, then the row statistics if the caller keeps none
  const size_t bb = (bounds_bytes(B) + 255) & ~size_t(255);
  char *tmp = nullptr;
  if ((rc = scratch_alloc(reinterpret_cast<void **>(&tmp), bb + (row_ws ? 0 : (size_t)chunk->n_rows * 4 * sizeof(float)), st)) !=
      FOPD_OK)
    return rc;
  unsigned long long *bounds = reinterpret_cast<unsigned long long *>(tmp);
  float *ws = row_ws ? row_ws : reinterpret_cast<float *>(tmp + bb);
  rc = launch_stats(chunk, B, lp_s, lp_t, kl, ratio, ws, status, st);
  if (rc == FOPD_OK) rc = launch_sample_bounds(chunk->sample_id, chunk->n_rows, B, bounds, st);
  if (rc == FOPD_OK) {
    segment_reduce_kernel<<<B, kSegThreads, 0, st>>>(to_dev(chunk), B, ws, nullptr, 0, bounds_or_null(bounds, B), acc);
    rc = launch_ok();
  }
  if (cudaFreeAsync(tmp, st) != cudaSuccess) rc = FOPD_ERR_CUDA;
  return rc;
}

int fopd_token_stats_student(const fopd_chunk *chunk, int32_t B, float *lp_s, float *ratio, double *acc,
                             int32_t *status, void *stream) {
  int rc = check_chunk(chunk, B, false);
  if (rc != FOPD_OK) return rc;
  if (!acc) return FOPD_ERR_NULL;
  if (chunk->n_rows == 0) return FOPD_OK;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t bb = (bounds_bytes(B) + 255) & ~size_t(255);
  char *tmp = nullptr;
  if ((rc = scratch_alloc(reinterpret_cast<void **>(&tmp), bb + (size_t)chunk->n_rows * 4 * sizeof(float), st)) != FOPD_OK)
    return rc;
  unsigned long long *bounds = reinterpret_cast<unsigned long long *>(tmp);
  float *ws = reinterpret_cast<float *>(tmp + bb);
  const ChunkDev d = to_dev(chunk);
  const unsigned grid = row_grid(chunk->n_rows);
  const bool short_row = chunk->vocab / (chunk->dtype == FOPD_BF16 ? 8 : 4) < kShortRowVecs;
#define FOPD_LAUNCH_STUDENT(DT, T) token_stats_student_kernel<DT, T><<<grid, T, 0, st>>>(d, B, lp_s, ratio, ws, status)
  if (chunk->dtype == FOPD_BF16) {
    if (short_row) FOPD_LAUNCH_STUDENT(FOPD_BF16, kStatsThreadsShortRow);
    else FOPD_LAUNCH_STUDENT(FOPD_BF16, kStatsThreads);
  } else {
    if (short_row) FOPD_LAUNCH_STUDENT(FOPD_F32, kStatsThreadsShortRow);
    else FOPD_LAUNCH_STUDENT(FOPD_F32, kStatsThreads);
  }
#undef FOPD_LAUNCH_STUDENT
  rc = launch_ok();
  if (rc == FOPD_OK) rc = launch_sample_bounds(chunk->sample_id, chunk->n_rows, B, bounds, st);
  if (rc == FOPD_OK) {
    segment_reduce_kernel<<<B, kSegThreads, 0, st>>>(d, B, ws, nullptr, 0, bounds_or_null(bounds, B), acc);
    rc = launch_ok();
  }
  if (cudaFreeAsync(tmp, st) != cudaSuccess) rc = FOPD_ERR_CUDA;
  return rc;
}

int fopd_sample_freshness(const double *acc, const int32_t *staleness, const int32_t *seq_len,
                          const float *d_sup, int32_t B, fopd_params p, float *f, float *w,
                          float *d_roll, float *l_distill, float *m_align, float *coef,
                          float *buffer_means, int32_t *status, void *stream) {
  if (B <= 0) return FOPD_ERR_SIZE;
  if (!acc || !staleness || !seq_len || !coef) return FOPD_ERR_NULL;
  int rc = check_params(p);
  if (rc != FOPD_OK) return rc;
  freshness_kernel<<<1, 256, 0, static_cast<cudaStream_t>(stream)>>>(
      acc, staleness, seq_len, d_sup, B, p, f, w, d_roll, l_distill, m_align, coef, buffer_means, status);
  return launch_ok();
}

int fopd_loss_fwd_bwd(const fopd_chunk *chunk, int32_t B, const float *coef, const float *row_ws,
                      fopd_params p, void *dlogits, double *loss_acc, int32_t *status, void *stream) {
  int rc = check_chunk(chunk, B);
  if (rc != FOPD_OK) return rc;
  if ((rc = check_params(p)) != FOPD_OK) return rc;
  if (!coef || !loss_acc) return FOPD_ERR_NULL;
  if (chunk->n_rows == 0) return FOPD_OK;
  if (!dlogits) return FOPD_ERR_NULL;
  if (!aligned16(dlogits) || (row_ws && !aligned16(row_ws))) return FOPD_ERR_ALIGN;
  {
    const int64_t esz = chunk->dtype == FOPD_BF16 ? 2 : 4;
    const uintptr_t bytes = (uintptr_t)(chunk->n_rows * chunk->row_stride * esz);
    const uintptr_t o = (uintptr_t)dlogits, s = (uintptr_t)chunk->student, t = (uintptr_t)chunk->teacher;
    if ((o < s + bytes && s < o + bytes) || (o < t + bytes && t < o + bytes)) return FOPD_ERR_ALIAS;
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const ChunkDev d = to_dev(chunk);
  const float *ws = row_ws;
  // one temporary: the samples' row ranges, then (without cached statistics) [n_rows, 4] row
  // statistics and [n_rows] row weights
  const size_t bb = (bounds_bytes(B) + 255) & ~size_t(255);
  char *blk = nullptr;
  if ((rc = scratch_alloc(reinterpret_cast<void **>(&blk), bb + (ws ? 0 : (size_t)chunk->n_rows * 5 * sizeof(float)), st)) !=
      FOPD_OK)
    return rc;
  unsigned long long *bounds = reinterpret_cast<unsigned long long *>(blk);
  bool grad_done = false;
  if (!ws) {
    // No cached statistics.  Preferred: the on-chip kernel, which forms the sums and the
    // gradient of a row while it is on chip and leaves the row statistics in tmp.  Shapes it
    // cannot take fall back to the statistics sweep + streaming gradient pair.
    float *tmp = reinterpret_cast<float *>(blk + bb);
    ws = tmp;
    // (the sampled-token form needs no teacher row for its gradient: statistics sweep + one pass)
    rc = chunk->loss_kind != FOPD_LOSS_FULL_KL
             ? kNotApplicable
             : chunk->dtype == FOPD_BF16 ? launch_fused<FOPD_BF16>(chunk, B, coef, p.lambda, dlogits, tmp, status, st)
                                         : launch_fused<FOPD_F32>(chunk, B, coef, p.lambda, dlogits, tmp, status, st);
    if (rc == FOPD_OK) grad_done = true;
    else if (rc == kNotApplicable)
      rc = launch_stats(chunk, B, nullptr, nullptr, nullptr, nullptr, tmp, status, st);
  }
  if (rc == FOPD_OK && !grad_done) {
    const unsigned grid = row_grid(chunk->n_rows);
    const bool short_row = chunk->vocab / (chunk->dtype == FOPD_BF16 ? 8 : 4) < kShortRowVecs;
#define FOPD_LAUNCH_GRAD(DT, T, TS)                                                      \
  do {                                                                                     \
    if (chunk->loss_kind == FOPD_LOSS_SAMPLED_KL)                                          \
      grad_sampled_kernel<DT, TS><<<grid, TS, 0, st>>>(d, B, coef, ws, p.lambda, dlogits); \
    else                                                                                   \
      grad_stream_kernel<DT, T><<<grid, T, 0, st>>>(d, B, coef, ws, p.lambda, dlogits);    \
  } while (0)
    if (chunk->dtype == FOPD_BF16) {
      if (short_row) FOPD_LAUNCH_GRAD(FOPD_BF16, kGradThreadsShortRow, kSampledThreadsShortRow);
      else FOPD_LAUNCH_GRAD(FOPD_BF16, kGradThreads, kSampledThreads);
    } else {
      if (short_row) FOPD_LAUNCH_GRAD(FOPD_F32, kGradThreadsShortRow, kSampledThreadsShortRow);
      else FOPD_LAUNCH_GRAD(FOPD_F32, kGradThreads, kSampledThreads);
    }
#undef FOPD_LAUNCH_GRAD
    rc = launch_ok();
  }
  if (rc == FOPD_OK) rc = launch_sample_bounds(chunk->sample_id, chunk->n_rows, B, bounds, st);
  if (rc == FOPD_OK) {
    segment_reduce_kernel<<<B, kSegThreads, 0, st>>>(d, B, ws, coef, 1, bounds_or_null(bounds, B), loss_acc);
    rc = launch_ok();
  }
  if (cudaFreeAsync(blk, st) != cudaSuccess) rc = FOPD_ERR_CUDA;
  return rc;
}

int fopd_loss_fwd_bwd_plan(int32_t dtype, int64_t vocab, int32_t *cluster_size, int32_t *block_threads,
                           int32_t *resident_clusters, int32_t *smem_bytes) {
  if (dtype != FOPD_BF16 && dtype != FOPD_F32) return FOPD_ERR_DTYPE;
  if (vocab <= 0 || vocab > (int64_t)1 << 30) return FOPD_ERR_SIZE;
  FusedPlan plan;
  const int64_t nvec = vocab / (dtype == FOPD_BF16 ? 8 : 4);
  int rc = FOPD_OK;
  if (nvec >= 1) rc = dtype == FOPD_BF16 ? fused_plan<FOPD_BF16>(nvec, &plan) : fused_plan<FOPD_F32>(nvec, &plan);
  if (rc != FOPD_OK) return rc;
  if (cluster_size) *cluster_size = plan.cluster;
  if (block_threads) *block_threads = plan.cluster ? plan.warps * 32 + 32 : 0;
  if (resident_clusters) *resident_clusters = plan.max_clusters;
  if (smem_bytes) *smem_bytes = (int32_t)plan.smem;
  return FOPD_OK;
}

int fopd_loss_fwd_bwd_set_plan(int32_t dtype, int64_t vocab, int32_t cluster_size) {
  if (dtype != FOPD_BF16 && dtype != FOPD_F32) return FOPD_ERR_DTYPE;
  if (vocab <= 0 || vocab > (int64_t)1 << 30 || cluster_size > kMaxClusterSize) return FOPD_ERR_SIZE;
  const int64_t nvec = vocab / (dtype == FOPD_BF16 ? 8 : 4);
  if (nvec < 1) return cluster_size > 0 ? FOPD_ERR_SIZE : FOPD_OK;
  const int pin = cluster_size < 0 ? -1 : cluster_size;
  FusedPlan plan;
  std::lock_guard<std::mutex> lock(g_fused_mu);
  int rc = dtype == FOPD_BF16 ? make_fused_plan<FOPD_BF16>(nvec, pin, &plan) : make_fused_plan<FOPD_F32>(nvec, pin, &plan);
  if (rc != FOPD_OK) return rc;
  if (pin > 0 && !plan.cluster) return FOPD_ERR_SIZE;  // that cluster size cannot hold the row on this device
  PlanEntry *e = plan_entry(dtype, nvec);
  if (!e) return FOPD_ERR_CUDA;
  e->pin = pin;
  e->plan = plan;
  e->planned = true;
  return FOPD_OK;
}

int fopd_selftest_bounded_wait(int64_t limit_cycles, int32_t *status, int64_t *waited_cycles, void *stream) {
  if (!status) return FOPD_ERR_NULL;
  if (limit_cycles < 0 || limit_cycles > kWaitCycles) return FOPD_ERR_SIZE;
  bounded_wait_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(
      (long long)limit_cycles, status, reinterpret_cast<long long *>(waited_cycles));
  return launch_ok();
}

int fopd_release_device_memory(void) {
  int rc = scratch_release();
  const int rc2 = host_step_release();
  return rc != FOPD_OK ? rc : rc2;
}

int fopd_loss_finalize(const double *loss_acc, const double *acc, const float *w, int32_t B,
                       fopd_params p, float *per_sample_loss, float *loss_out, void *stream) {
  if (B <= 0) return FOPD_ERR_SIZE;
  if (!loss_acc || !acc || !w || !loss_out) return FOPD_ERR_NULL;
  int rc = check_params(p);
  if (rc != FOPD_OK) return rc;
  finalize_kernel<<<1, 256, 0, static_cast<cudaStream_t>(stream)>>>(loss_acc, acc, w, B, p.lambda,
                                                                    per_sample_loss, loss_out);
  return launch_ok();
}

int fopd_check_status(const int32_t *status, int32_t *bits_out, void *stream) {
  if (!status) return FOPD_ERR_NULL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int32_t bits = 0;
  if (cudaMemcpyAsync(&bits, status, sizeof(bits), cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return FOPD_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return FOPD_ERR_CUDA;
  if (bits_out) *bits_out = bits;
  return bits == 0 ? FOPD_OK : FOPD_ERR_DEVICE;
}

}  // extern "C"
