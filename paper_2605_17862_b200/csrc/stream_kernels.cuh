// Streaming kernels of libfopd that work for any vocabulary size and both
// logit dtypes: the statistics sweep, the single-pass gradient sweep that uses
// cached row statistics, the per-sample segmented reduction, freshness and
// the final loss.  One CTA per row (the grid is the row count: the hardware's
// block scheduler balances rows of unequal cost and staggers the CTAs' position
// in their rows, which measured 5-9 % faster than persistent CTAs in lock step);
// rows are 16-byte aligned so the body uses 16-byte loads and a scalar tail
// covers vocabularies that do not fill the last vector.
#pragma once

#include "common.cuh"

namespace fopd {

// Block sizes by row length (measured): the statistics sweep, bound by the special-function
// pipe, wants many small CTAs per SM; the gradient sweep, bound by memory, one large one for long
// rows.  Short rows take small blocks so that more CTAs overlap their start-up (bf16 rows of
// 32,000: gradient sweep 6.4-6.8 TB/s with 256 threads against 6.3-6.4 with 512).
constexpr int kStatsThreads = 256, kStatsThreadsShortRow = 128;
constexpr int kGradThreads = 1024, kGradThreadsShortRow = 256;
// the sampled-token gradient sweep (one read, one write per element) wants more CTAs per SM in flight
constexpr int kSampledThreads = 512, kSampledThreadsShortRow = 256;
constexpr int64_t kShortRowVecs = 8192;  // rows of fewer 16-byte vectors count as short
constexpr int kUnroll = 4;
constexpr int64_t kMaxGrid = 1 << 30;

struct ChunkDev {
  const void *student, *teacher;
  const float *behav;
  const int32_t *tokens;
  const uint8_t *mask;
  const int32_t *sid;
  int64_t n_rows, vocab, stride;
  int kind;  // fopd_loss_kind
};

// Is row n aligned (counts towards U_i)?  Records bad ids in the status word.
__device__ __forceinline__ bool row_is_aligned(const ChunkDev &c, int64_t n, int32_t B,
                                               int32_t *status, bool report) {
  // three independent loads, issued together: a CTA's first logits load waits for one memory
  // round trip, not for a chain of them (tokens[n] is read for masked rows too; it is not used)
  const int32_t sid = c.sid[n], y = c.tokens[n];
  const uint8_t m = c.mask[n];
  bool ok = true;
  if (sid < 0 || sid >= B) {
    if (report && status) atomicOr(status, FOPD_DEV_BAD_SAMPLE);
    ok = false;
  }
  if (m == 0) return false;
  if (y < 0 || y >= c.vocab) {
    if (report && status) atomicOr(status, FOPD_DEV_BAD_TOKEN);
    ok = false;
  }
  return ok;
}

// Turns the finished accumulators of a row into the quantities of Sec. 4.1 /
// Eq. 10 / Eq. 12 and writes the per-row outputs.  Called by one thread.
template <int DT>
__device__ __forceinline__ void finish_row(int64_t n, const RowAcc &r, float sy, float ty, float b, int kind,
                                           float *lp_s, float *lp_t, float *kl_out, float *ratio, float *row_ws) {
  // log of the partition sums in full precision (logf, not the fast intrinsic)
  // differences are formed from the maxima and the logs separately, so that they do not inherit
  // the rounding of a large log-normaliser
  const float gs = logf(r.zs), gt = logf(r.zt);
  const float ls = r.ms + gs, lt = r.mt + gt;
  const float kl = r.as / r.zs - ((r.ms - r.mt) + (gs - gt));
  const float lps = (sy - r.ms) - gs, lpt = (ty - r.mt) - gt;
  const float d = lps - b;
  if (lp_s) lp_s[n] = lps;
  if (lp_t) lp_t[n] = lpt;
  const float rho = expf(d);  // fp32 is ample for the reported ratio; the drift integrand is formed in fp64 from d
  // sampled-token form of Eq. 12's loss: rho (lp_s - lp_t) on the stored token; the workspace
  // keeps the log-ratio, which the gradient takes as a constant
  const float log_ratio = lps - lpt;
  if (kl_out) kl_out[n] = kind == FOPD_LOSS_SAMPLED_KL ? rho * log_ratio : kl;
  if (ratio) ratio[n] = rho;
  reinterpret_cast<float4 *>(row_ws)[n] = make_float4(ls, lt, kind == FOPD_LOSS_SAMPLED_KL ? log_ratio : kl, d);
}

__device__ __forceinline__ void zero_row_outputs(int64_t n, float *lp_s, float *lp_t, float *kl_out,
                                                 float *ratio, float *row_ws) {
  if (lp_s) lp_s[n] = 0.f;
  if (lp_t) lp_t[n] = 0.f;
  if (kl_out) kl_out[n] = 0.f;
  if (ratio) ratio[n] = 0.f;
  reinterpret_cast<float4 *>(row_ws)[n] = make_float4(0.f, 0.f, 0.f, 0.f);
}

// Sweep one row from global memory into a per-thread RowAcc.
template <int DT, int kThreads>
__device__ __forceinline__ RowAcc sweep_row_global(const void *srow, const void *trow, int64_t V) {
  using E = Elem<DT>;
  constexpr int P = E::kPerVec;
  RowSweep acc;
  acc.init();
  const int64_t nvec = V / P;
  const uint4 *s4 = reinterpret_cast<const uint4 *>(srow);
  const uint4 *t4 = reinterpret_cast<const uint4 *>(trow);
  int64_t i = threadIdx.x;
  for (; i + (kUnroll - 1) * kThreads < nvec; i += kUnroll * kThreads) {
    uint4 a[kUnroll], b[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      a[u] = ld_stream(s4 + i + u * kThreads);
      b[u] = ld_stream(t4 + i + u * kThreads);
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      float s[P], t[P];
      E::unpack(a[u], s);
      E::unpack(b[u], t);
      acc.add<P>(s, t);
    }
  }
  for (; i < nvec; i += kThreads) {
    float s[P], t[P];
    E::unpack(ld_stream(s4 + i), s);
    E::unpack(ld_stream(t4 + i), t);
    acc.add<P>(s, t);
  }
  const int64_t tail = nvec * P + threadIdx.x;
  if (tail < V) acc.add1(E::load1(srow, tail), E::load1(trow, tail));
  return acc.settle();
}

// a1-a4: statistics sweep.  grid = rows (any grid works), block = kThreads.
template <int DT, int kThreads>
__global__ void __launch_bounds__(kThreads, 1024 / kThreads)
    token_stats_kernel(ChunkDev c, int32_t B, float *lp_s, float *lp_t, float *kl, float *ratio,
                       float *row_ws, int32_t *status) {
  using E = Elem<DT>;
  __shared__ RowAcc scratch[2][kThreads / 32];  // alternating per row: no barrier after the row's finish
  int par = 0;
  for (int64_t n = blockIdx.x; n < c.n_rows; n += gridDim.x) {
    if (!row_is_aligned(c, n, B, status, threadIdx.x == 0)) {
      if (threadIdx.x == 0) zero_row_outputs(n, lp_s, lp_t, kl, ratio, row_ws);
      continue;
    }
    // gathers of the stored token and its behaviour log-prob: issued now, used after the sweep
    float sy = 0.f, ty = 0.f, b = 0.f;
    if (threadIdx.x == 0) {
      const int32_t y = c.tokens[n];
      sy = E::load1(c.student, n * c.stride + y);
      ty = E::load1(c.teacher, n * c.stride + y);
      b = c.behav[n];
    }
    const char *srow = reinterpret_cast<const char *>(c.student) + n * c.stride * E::kBytes;
    const char *trow = reinterpret_cast<const char *>(c.teacher) + n * c.stride * E::kBytes;
    RowAcc acc = sweep_row_global<DT, kThreads>(srow, trow, c.vocab);
    acc = block_reduce<kThreads>(acc, scratch[par]);
    if (threadIdx.x == 0) finish_row<DT>(n, acc, sy, ty, b, c.kind, lp_s, lp_t, kl, ratio, row_ws);
    par ^= 1;
  }
}

// Student-only statistics sweep: what the first loop of Algorithm 1 needs (Eq. 10, Eq. 11: the
// rollout drift and the freshness depend on the student's and the behaviour policy's
// log-probabilities of the stored tokens alone).  One read of the student row, one ex2 per logit;
// the exponent is formed as in RowSweep.  row_ws gets {lse_s, 0, 0, d}: enough for the
// per-sample sums, not for the gradient sweep.
template <int DT, int kThreads>
__device__ __forceinline__ RowAcc sweep_row_student(const void *srow, int64_t V) {
  using E = Elem<DT>;
  constexpr int P = E::kPerVec;
  float ms = kNegBig, cs = kNegBig, zs = 0.f;
  auto add = [&](const float *s, int n) {
    float vs = s[0];
    for (int i = 1; i < n; ++i) vs = fmaxf(vs, s[i]);
    if (vs > ms) {
      const float cn = vs * kLog2e;
      zs *= ex2(cs - cn);
      ms = vs;
      cs = cn;
    }
    for (int i = 0; i < n; ++i) zs += ex2(fmaf(s[i], kLog2e, -cs));
  };
  const int64_t nvec = V / P;
  const uint4 *s4 = reinterpret_cast<const uint4 *>(srow);
  int64_t i = threadIdx.x;
  constexpr int kU = 2 * kUnroll;  // half the loads per vector of the two-row sweep: twice the vectors in flight
  for (; i + (kU - 1) * kThreads < nvec; i += kU * kThreads) {
    uint4 a[kU];
#pragma unroll
    for (int u = 0; u < kU; ++u) a[u] = ld_stream(s4 + i + u * kThreads);
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      float s[P];
      E::unpack(a[u], s);
      add(s, P);
    }
  }
  for (; i < nvec; i += kThreads) {
    float s[P];
    E::unpack(ld_stream(s4 + i), s);
    add(s, P);
  }
  const int64_t tail = nvec * P + threadIdx.x;
  if (tail < V) {
    const float s1 = E::load1(srow, tail);
    add(&s1, 1);
  }
  RowAcc r;
  r.init();
  r.ms = ms;
  r.zs = __fmaf_rn(zs, -fmaf(ms, kLog2e, -cs) * kLn2, zs);  // the rounding of the scaled maximum, taken out
  return r;
}

template <int DT, int kThreads>
__global__ void __launch_bounds__(kThreads, 1024 / kThreads)
    token_stats_student_kernel(ChunkDev c, int32_t B, float *lp_s, float *ratio, float *row_ws, int32_t *status) {
  using E = Elem<DT>;
  __shared__ RowAcc scratch[2][kThreads / 32];  // alternating per row: no barrier after the row's finish
  int par = 0;
  for (int64_t n = blockIdx.x; n < c.n_rows; n += gridDim.x) {
    if (!row_is_aligned(c, n, B, status, threadIdx.x == 0)) {
      if (threadIdx.x == 0) zero_row_outputs(n, lp_s, nullptr, nullptr, ratio, row_ws);
      continue;
    }
    float sy = 0.f, b = 0.f;
    if (threadIdx.x == 0) {
      sy = E::load1(c.student, n * c.stride + c.tokens[n]);
      b = c.behav[n];
    }
    RowAcc acc = sweep_row_student<DT, kThreads>(reinterpret_cast<const char *>(c.student) + n * c.stride * E::kBytes, c.vocab);
    acc = block_reduce<kThreads>(acc, scratch[par]);
    if (threadIdx.x == 0) {
      const float gs = logf(acc.zs);
      const float lps = (sy - acc.ms) - gs, d = lps - b;
      if (lp_s) lp_s[n] = lps;
      if (ratio) ratio[n] = expf(d);
      reinterpret_cast<float4 *>(row_ws)[n] = make_float4(acc.ms + gs, 0.f, 0.f, d);
    }
    par ^= 1;
  }
}

// Per-row constants of the gradient sweep (see fopd_loss_fwd_bwd):
//   dS_v = cp_v * ((s_v - t_v) - K) + [v == y] * cg
//   cp_v = coef * p_s(v) = 2^(s_v*log2e + e0),  e0 = log2(coef) - lse_s*log2e
//   K    = kl + g + (lse_s - lse_t),  g = lambda * rho * d,  cg = coef * g
struct GradRow {
  float e0, K, cg;
  int32_t y;
};

__device__ __forceinline__ GradRow make_grad_row(float4 ws, float coef, float lambda, int32_t y) {
  const float d = ws.w;
  const float g = lambda * (expf(d) * d);  // lambda * rho * d, the derivative of lambda * k3
  GradRow r;
  r.e0 = log2f(coef) - ws.x * kLog2e;
  r.K = ws.z + g + (ws.x - ws.y);
  r.cg = coef * g;
  r.y = y;
  return r;
}

// Gradient of one vector without the stored token's extra term (added afterwards by
// the thread that wrote the token's vector).
template <int DT>
__device__ __forceinline__ uint4 grad_vec(const uint4 &sv, const uint4 &tv, const GradRow &r) {
  using E = Elem<DT>;
  constexpr int P = E::kPerVec;
  float s[P], t[P], o[P];
  E::unpack(sv, s);
  E::unpack(tv, t);
#pragma unroll
  for (int i = 0; i < P; ++i) o[i] = ex2(fmaf(s[i], kLog2e, r.e0)) * ((s[i] - t[i]) - r.K);
  return E::pack(o);
}

// A row that is not differentiated (masked, padded, bad id, gated or invalid sample): +0.
template <int DT, int kThreads>
__device__ __forceinline__ void zero_fill_row(char *orow, int64_t V) {
  using E = Elem<DT>;
  constexpr int P = E::kPerVec;
  const int64_t nvec = V / P;
  uint4 *o4 = reinterpret_cast<uint4 *>(orow);
  const uint4 z = make_uint4(0u, 0u, 0u, 0u);
  for (int64_t i = threadIdx.x; i < nvec; i += kThreads) st_stream(o4 + i, z);
  const int64_t tail = nvec * P + threadIdx.x;
  if (tail < V) E::store1(orow, tail, 0.f);
}

// One streaming pass over a differentiated row: read S, read T, write dS.  r.y is the stored
// token's column within this row view (any value outside [0, V) when it lies elsewhere).
template <int DT, int kThreads>
__device__ __forceinline__ void grad_row_sweep(const char *srow, const char *trow, char *orow, int64_t V,
                                               const GradRow &r) {
  using E = Elem<DT>;
  constexpr int P = E::kPerVec;
  const int64_t nvec = V / P;
  const uint4 *s4 = reinterpret_cast<const uint4 *>(srow);
  const uint4 *t4 = reinterpret_cast<const uint4 *>(trow);
  uint4 *o4 = reinterpret_cast<uint4 *>(orow);
  int64_t i = threadIdx.x;
  for (; i + (kUnroll - 1) * kThreads < nvec; i += kUnroll * kThreads) {
    uint4 a[kUnroll], b[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      a[u] = ld_stream(s4 + i + u * kThreads);
      b[u] = ld_stream(t4 + i + u * kThreads);
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) st_stream(o4 + i + u * kThreads, grad_vec<DT>(a[u], b[u], r));
  }
  for (; i < nvec; i += kThreads) st_stream(o4 + i, grad_vec<DT>(ld_stream(s4 + i), ld_stream(t4 + i), r));
  // the stored token's element: rewritten with its extra term by the thread that stored its
  // vector (one thread, so the two stores to that address stay in order)
  const int64_t yv = r.y / P;
  if (r.y >= 0 && yv < nvec && (int)(yv % kThreads) == (int)threadIdx.x) {
    const float s = E::load1(srow, r.y), t = E::load1(trow, r.y);
    E::store1(orow, r.y, fmaf(ex2(fmaf(s, kLog2e, r.e0)), (s - t) - r.K, r.cg));
  }
  const int64_t tail = nvec * P + threadIdx.x;
  if (tail < V) {
    const float s = E::load1(srow, tail), t = E::load1(trow, tail);
    float o = ex2(fmaf(s, kLog2e, r.e0)) * ((s - t) - r.K);
    if (tail == r.y) o += r.cg;
    E::store1(orow, tail, o);
  }
}

// a8 with cached row statistics: one streaming pass, read S, read T, write dS.
// grid = rows (any grid works), block = kThreads.
template <int DT, int kThreads>
__global__ void __launch_bounds__(kThreads, 1024 / kThreads)
    grad_stream_kernel(ChunkDev c, int32_t B, const float *coef, const float *row_ws, float lambda,
                       void *dlogits) {
  using E = Elem<DT>;
  for (int64_t n = blockIdx.x; n < c.n_rows; n += gridDim.x) {
    char *orow = reinterpret_cast<char *>(dlogits) + n * c.stride * E::kBytes;
    // independent loads first (side arrays and cached statistics), then the one that depends
    // on them (the sample's weight): two memory round trips before the first logits load
    const int32_t sid = c.sid[n], y = c.tokens[n];
    const uint8_t m = c.mask[n];
    const float4 ws = reinterpret_cast<const float4 *>(row_ws)[n];
    const bool sid_ok = sid >= 0 && sid < B;
    float cf = sid_ok ? coef[sid] : 0.f;
    if (m == 0 || y < 0 || y >= c.vocab) cf = 0.f;
    if (!(cf > 0.f)) {
      zero_fill_row<DT, kThreads>(orow, c.vocab);
      continue;
    }
    const GradRow r = make_grad_row(ws, cf, lambda, y);
    grad_row_sweep<DT, kThreads>(reinterpret_cast<const char *>(c.student) + n * c.stride * E::kBytes,
                                 reinterpret_cast<const char *>(c.teacher) + n * c.stride * E::kBytes, orow, c.vocab,
                                 r);
  }
}

// Row range of every sample within a chunk, found in one pass over the rows: bounds[2i] =
// first row whose sample id is i, bounds[2i + 1] = one past the last such row (first >= last:
// the sample has no row in this chunk).  Rows of a sample are contiguous, so a row starts a
// run where its id differs from the row before and ends one where it differs from the row
// after; minimum / maximum over the runs keep the result unique when an out-of-range id sits
// in the middle of a sample (the rows in between are skipped by their own id).
static __global__ void __launch_bounds__(256) sample_bounds_init_kernel(int32_t B, unsigned long long *bounds) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < B) {
    bounds[2 * i] = ~0ull;
    bounds[2 * i + 1] = 0ull;
  }
}
static __global__ void __launch_bounds__(256)
    sample_bounds_kernel(const int32_t *sid, int64_t n_rows, int32_t B, unsigned long long *bounds) {
  const int64_t n = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (n >= n_rows) return;
  const int32_t s = sid[n];
  if (s < 0 || s >= B) return;
  if (n == 0 || sid[n - 1] != s) atomicMin(&bounds[2 * (int64_t)s], (unsigned long long)n);
  if (n == n_rows - 1 || sid[n + 1] != s) atomicMax(&bounds[2 * (int64_t)s + 1], (unsigned long long)(n + 1));
}

// a8 for the sampled-token form of the loss, with cached row statistics: one streaming pass
// that reads S and writes dS.  For a differentiated row
//   dS_v = coef rho (r + lambda d) (1[v = y] - p_s(v)),   r = lp_s - lp_t (constant), d = lp_s - b,
// i.e. -G cp_v + [v == y] G coef with cp_v = coef p_s(v) = 2^(s_v*log2e + e0), G = rho (r + lambda d).
template <int DT, int kThreads>
__global__ void __launch_bounds__(kThreads, 1024 / kThreads)
    grad_sampled_kernel(ChunkDev c, int32_t B, const float *coef, const float *row_ws, float lambda, void *dlogits) {
  using E = Elem<DT>;
  constexpr int P = E::kPerVec;
  for (int64_t n = blockIdx.x; n < c.n_rows; n += gridDim.x) {
    char *orow = reinterpret_cast<char *>(dlogits) + n * c.stride * E::kBytes;
    const int32_t sid = c.sid[n], y = c.tokens[n];
    const uint8_t m = c.mask[n];
    const float4 ws = reinterpret_cast<const float4 *>(row_ws)[n];
    const bool sid_ok = sid >= 0 && sid < B;
    float cf = sid_ok ? coef[sid] : 0.f;
    if (m == 0 || y < 0 || y >= c.vocab) cf = 0.f;
    if (!(cf > 0.f)) {
      zero_fill_row<DT, kThreads>(orow, c.vocab);
      continue;
    }
    const float d = ws.w, G = expf(d) * (ws.z + lambda * d);
    const float e0 = log2f(cf) - ws.x * kLog2e, negG = -G, cg = cf * G;
    const char *srow = reinterpret_cast<const char *>(c.student) + n * c.stride * E::kBytes;
    const int64_t V = c.vocab, nvec = V / P;
    const uint4 *s4 = reinterpret_cast<const uint4 *>(srow);
    uint4 *o4 = reinterpret_cast<uint4 *>(orow);
    auto one = [&](const uint4 &sv) {
      float s[P], o[P];
      E::unpack(sv, s);
#pragma unroll
      for (int i = 0; i < P; ++i) o[i] = ex2(fmaf(s[i], kLog2e, e0)) * negG;
      return E::pack(o);
    };
    int64_t i = threadIdx.x;
    for (; i + (kUnroll - 1) * kThreads < nvec; i += kUnroll * kThreads) {
      uint4 a[kUnroll];
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) a[u] = ld_stream(s4 + i + u * kThreads);
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) st_stream(o4 + i + u * kThreads, one(a[u]));
    }
    for (; i < nvec; i += kThreads) st_stream(o4 + i, one(ld_stream(s4 + i)));
    // the stored token's element: rewritten with its extra term by the thread that stored its vector
    const int64_t yv = y / P;
    if (yv < nvec && (int)(yv % kThreads) == (int)threadIdx.x) {
      const float s = E::load1(srow, y);
      E::store1(orow, y, fmaf(ex2(fmaf(s, kLog2e, e0)), negG, cg));
    }
    const int64_t tail = nvec * P + threadIdx.x;
    if (tail < V) {
      const float s = E::load1(srow, tail);
      float o = ex2(fmaf(s, kLog2e, e0)) * negG;
      if (tail == y) o = fmaf(ex2(fmaf(s, kLog2e, e0)), negG, cg);
      E::store1(orow, tail, o);
    }
  }
}

// The same range for one sample, found by the block that reduces it (all threads scan the
// chunk's ids together; shared-memory minimum / maximum over the runs).  Costs a pass over the
// ids per sample, which is what a batch of a few samples wants: no extra launches.
constexpr int32_t kFewSamples = 32;
__device__ __forceinline__ void sample_row_range(const int32_t *sid, int64_t n_rows, int32_t key,
                                                 unsigned long long *range_sh, unsigned long long &lo,
                                                 unsigned long long &hi) {
  if (threadIdx.x == 0) {
    range_sh[0] = ~0ull;
    range_sh[1] = 0ull;
  }
  __syncthreads();
  for (int64_t n = threadIdx.x; n < n_rows; n += blockDim.x) {
    if (sid[n] != key) continue;
    if (n == 0 || sid[n - 1] != key) atomicMin(&range_sh[0], (unsigned long long)n);
    if (n == n_rows - 1 || sid[n + 1] != key) atomicMax(&range_sh[1], (unsigned long long)(n + 1));
  }
  __syncthreads();
  lo = range_sh[0];
  hi = range_sh[1];
}

// a5: deterministic segmented reduction of per-row statistics into per-sample
// sums.  One block per sample over the sample's row range (from `bounds`, or found here when
// bounds is NULL); every thread sums a
// fixed strided subset in fp64 and a fixed tree combines them, so a rerun
// reproduces the bits.  mode 0: acc[B,4] += {cnt, sum k3, sum kl, rows}.
// mode 1: loss_acc[B,2] += {sum kl, sum k3} over rows of samples with coef > 0.
constexpr int kSegThreads = 1024;

static __global__ void __launch_bounds__(kSegThreads)
    segment_reduce_kernel(ChunkDev c, int32_t B, const float *row_ws, const float *coef, int mode,
                          const unsigned long long *bounds, double *out) {
  __shared__ double sh[3][kSegThreads];
  __shared__ unsigned long long range_sh[2];
  const int32_t i = blockIdx.x;
  if (mode == 1 && !(coef[i] > 0.f)) return;
  unsigned long long lo_u, hi_u;
  if (bounds) {
    lo_u = bounds[2 * (int64_t)i];
    hi_u = bounds[2 * (int64_t)i + 1];
  } else {
    sample_row_range(c.sid, c.n_rows, i, range_sh, lo_u, hi_u);
  }
  if (lo_u >= hi_u) return;
  const int64_t lo = (int64_t)lo_u, hi = (int64_t)hi_u;
  double cnt = 0.0, sk3 = 0.0, skl = 0.0;
  for (int64_t n = lo + threadIdx.x; n < hi; n += kSegThreads) {
    if (c.sid[n] != i || c.mask[n] == 0) continue;
    const int32_t y = c.tokens[n];
    if (y < 0 || y >= c.vocab) continue;
    const float4 ws = reinterpret_cast<const float4 *>(row_ws)[n];
    const double d = (double)ws.w;
    cnt += 1.0;
    const double rho = exp(d);
    sk3 += rho * d - expm1(d);  // rho log rho - (rho - 1), Eq. 10 integrand
    skl += c.kind == FOPD_LOSS_SAMPLED_KL ? rho * (double)ws.z : (double)ws.z;  // token loss of Eq. 12 in the chunk's form
  }
  sh[0][threadIdx.x] = cnt;
  sh[1][threadIdx.x] = sk3;
  sh[2][threadIdx.x] = skl;
  __syncthreads();
  for (int off = kSegThreads / 2; off > 0; off >>= 1) {
    if (threadIdx.x < off) {
      sh[0][threadIdx.x] += sh[0][threadIdx.x + off];
      sh[1][threadIdx.x] += sh[1][threadIdx.x + off];
      sh[2][threadIdx.x] += sh[2][threadIdx.x + off];
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    if (mode == 0) {
      double *a = out + 4 * (int64_t)i;
      a[FOPD_ACC_CNT] += sh[0][0];
      a[FOPD_ACC_K3] += sh[1][0];
      a[FOPD_ACC_KL] += sh[2][0];
      a[FOPD_ACC_ROWS] += (double)(hi - lo);
    } else {
      double *a = out + 2 * (int64_t)i;
      a[0] += sh[2][0];
      a[1] += sh[1][0];
    }
  }
}

// a6: freshness, gate, alignment ratio, per-token weight.  Single block.
static __global__ void __launch_bounds__(256)
    freshness_kernel(const double *acc, const int32_t *tau, const int32_t *H, const float *d_sup,
                     int32_t B, fopd_params p, float *f, float *w, float *d_roll, float *l_distill,
                     float *m_align, float *coef, float *buffer_means, int32_t *status) {
  __shared__ double sh[2][256];
  double sum_f = 0.0, sum_m = 0.0;
  for (int32_t i = threadIdx.x; i < B; i += 256) {
    const double cnt = acc[4 * (int64_t)i + FOPD_ACC_CNT];
    const int32_t t = tau[i], h = H[i];
    if (t < 0 && status) atomicOr(status, FOPD_DEV_BAD_TAU);
    if ((h <= 0 || cnt > (double)h) && status) atomicOr(status, FOPD_DEV_BAD_LENGTH);
    double fi = 0.0, wi = 0.0, dr = 0.0, li = 0.0, mi = 0.0, ci = 0.0;
    const double ds = d_sup ? (double)d_sup[i] : 0.0;
    // d_sup = +inf marks a sample with no aligned supervision position: invalid (Algorithm 1)
    if (cnt > 0.0 && h > 0 && t >= 0 && !isinf(ds)) {
      dr = acc[4 * (int64_t)i + FOPD_ACC_K3] / cnt;
      li = acc[4 * (int64_t)i + FOPD_ACC_KL] / cnt;
      const double surrogate = (double)p.alpha * sqrt(fmax(dr, 0.0)) + (double)p.beta * sqrt(fmax(ds, 0.0));
      fi = exp(-surrogate) / ((double)t + 1.0);
      wi = fmax(fi - (double)p.xi, 0.0);
      mi = cnt / (double)h;
      ci = wi / ((double)B * cnt);
    }
    if (f) f[i] = (float)fi;
    if (w) w[i] = (float)wi;
    if (d_roll) d_roll[i] = (float)dr;
    if (l_distill) l_distill[i] = (float)li;
    if (m_align) m_align[i] = (float)mi;
    coef[i] = (float)ci;
    sum_f += fi;
    sum_m += mi;
  }
  if (buffer_means) {
    sh[0][threadIdx.x] = sum_f;
    sh[1][threadIdx.x] = sum_m;
    __syncthreads();
    for (int off = 128; off > 0; off >>= 1) {
      if (threadIdx.x < off) {
        sh[0][threadIdx.x] += sh[0][threadIdx.x + off];
        sh[1][threadIdx.x] += sh[1][threadIdx.x + off];
      }
      __syncthreads();
    }
    if (threadIdx.x == 0) {
      buffer_means[0] = (float)(sh[0][0] / (double)B);
      buffer_means[1] = (float)(sh[1][0] / (double)B);
    }
  }
}

// a7: L_i = w_i (l_i + lambda D_roll_i), L = (1/B) sum_i L_i.  Single block.
static __global__ void __launch_bounds__(256)
    finalize_kernel(const double *loss_acc, const double *acc, const float *w, int32_t B, float lambda,
                    float *per_sample, float *loss_out) {
  __shared__ double sh[256];
  double s = 0.0;
  for (int32_t i = threadIdx.x; i < B; i += 256) {
    const double cnt = acc[4 * (int64_t)i + FOPD_ACC_CNT];
    double Li = 0.0;
    if (cnt > 0.0 && w[i] > 0.f)
      Li = (double)w[i] * (loss_acc[2 * (int64_t)i] + (double)lambda * loss_acc[2 * (int64_t)i + 1]) / cnt;
    if (per_sample) per_sample[i] = (float)Li;
    s += Li;
  }
  sh[threadIdx.x] = s;
  __syncthreads();
  for (int off = 128; off > 0; off >>= 1) {
    if (threadIdx.x < off) sh[threadIdx.x] += sh[threadIdx.x + off];
    __syncthreads();
  }
  if (threadIdx.x == 0) loss_out[0] = (float)(sh[0] / (double)B);
}

}  // namespace fopd
