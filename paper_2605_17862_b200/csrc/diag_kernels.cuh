// Diagnostics next to the loss path: the full-vocabulary KL between two logit
// tensors row by row (the supervision drift of Eq. 10 when they are the teacher
// under the current and under the stored context) with the entropy of the first
// distribution, their per-sample means, and the buffer-level refresh rule of
// Eq. 14-15.  Same streaming sweep as the statistics kernel; not on the timed
// hot path.
#pragma once

#include "stream_kernels.cuh"

namespace fopd {

constexpr int kDiagThreads = 256;

// Row accumulators for KL(p || q) and H(p): p-side max m, Z = sum e^{a-m},
// A = sum e^{a-m} (a - b), S = sum e^{a-m} (a - m); q-side max and Z.
//   KL = A / Z - lse_p + lse_q,   H(p) = lse_p - E_p[a] = log Z - S / Z.
// Exponents are formed as (x - max) * log2(e) and the entropy sum is kept relative to the
// maximum, so neither loses accuracy when the logits sit far from zero.
struct DivAcc {
  RowAcc r;
  float ss;  // sum e^{a-m} (a - m), relative to the same running maximum as r.zs
  __device__ __forceinline__ void init() {
    r.init();
    ss = 0.f;
  }
  template <int N>
  __device__ __forceinline__ void add(const float (&a)[N], const float (&b)[N]) {
    const float va = max_of<N>(a), vb = max_of<N>(b);
    if (va > r.ms) {
      // new maximum m': sum e^{a-m'} (a - m') = e^{m-m'} (S + (m - m') Z)
      const float f = ex2((r.ms - va) * kLog2e);
      ss = f * fmaf(r.ms - va, r.zs, ss);
      r.zs *= f;
      r.as *= f;
      r.ms = va;
    }
    if (vb > r.mt) {
      r.zt *= ex2((r.mt - vb) * kLog2e);
      r.mt = vb;
    }
#pragma unroll
    for (int i = 0; i < N; ++i) {
      const float da = a[i] - r.ms;
      const float ea = ex2(da * kLog2e);
      r.zs += ea;
      r.as = fmaf(ea, a[i] - b[i], r.as);
      ss = fmaf(ea, da, ss);
      r.zt += ex2((b[i] - r.mt) * kLog2e);
    }
  }
  __device__ __forceinline__ void merge(const DivAcc &o) {
    const float M = fmaxf(r.ms, o.r.ms);
    const float fa = ex2((r.ms - M) * kLog2e), fb = ex2((o.r.ms - M) * kLog2e);
    // both sums moved to the common maximum M before they are added
    ss = __fmaf_rn(__fmaf_rn(r.ms - M, r.zs, ss), fa, __fmul_rn(__fmaf_rn(o.r.ms - M, o.r.zs, o.ss), fb));
    r.merge(o.r);
  }
};

__device__ __forceinline__ DivAcc shfl_xor(const DivAcc &a, int lane_mask) {
  DivAcc o;
  o.r = shfl_xor(a.r, lane_mask);
  o.ss = __shfl_xor_sync(0xffffffffu, a.ss, lane_mask);
  return o;
}

// One CTA per row.  vals[n] = {kl, entropy} (zeros for rows with mask = 0 or a bad sample id).
template <int DT>
__global__ void __launch_bounds__(kDiagThreads, 4)
    row_divergence_kernel(const void *first, const void *second, const uint8_t *mask, const int32_t *sid,
                          int64_t n_rows, int64_t V, int64_t stride, int32_t B, float *kl_out, float *ent_out,
                          float2 *vals, int32_t *status) {
  using E = Elem<DT>;
  constexpr int P = E::kPerVec;
  constexpr int kWarps = kDiagThreads / 32;
  __shared__ DivAcc scratch[2][kWarps];
  int par = 0;
  for (int64_t n = blockIdx.x; n < n_rows; n += gridDim.x) {
    const int32_t s = sid[n];
    bool ok = mask[n] != 0;
    if (s < 0 || s >= B) {
      if (threadIdx.x == 0 && status) atomicOr(status, FOPD_DEV_BAD_SAMPLE);
      ok = false;
    }
    if (!ok) {
      if (threadIdx.x == 0) {
        if (kl_out) kl_out[n] = 0.f;
        if (ent_out) ent_out[n] = 0.f;
        vals[n] = make_float2(0.f, 0.f);
      }
      continue;
    }
    const char *arow = reinterpret_cast<const char *>(first) + n * stride * E::kBytes;
    const char *brow = reinterpret_cast<const char *>(second) + n * stride * E::kBytes;
    const uint4 *a4 = reinterpret_cast<const uint4 *>(arow), *b4 = reinterpret_cast<const uint4 *>(brow);
    const int64_t nvec = V / P;
    DivAcc acc;
    acc.init();
    for (int64_t i = threadIdx.x; i < nvec; i += kDiagThreads) {
      float a[P], b[P];
      E::unpack(ld_stream(a4 + i), a);
      E::unpack(ld_stream(b4 + i), b);
      acc.add<P>(a, b);
    }
    const int64_t tail = nvec * P + threadIdx.x;
    if (tail < V) {
      const float a[1] = {E::load1(arow, tail)}, b[1] = {E::load1(brow, tail)};
      acc.add<1>(a, b);
    }
    // fixed-order merge: lanes, then warps
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) acc.merge(shfl_xor(acc, off));
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) scratch[par][warp] = acc;
    __syncthreads();
    if (warp == 0) {
      DivAcc t;
      t.init();
      if (lane < kWarps) t = scratch[par][lane];
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) t.merge(shfl_xor(t, off));
      if (lane == 0) {
        const float gp = logf(t.r.zs), gq = logf(t.r.zt);
        const float kl = t.r.as / t.r.zs - ((t.r.ms - t.r.mt) + (gp - gq));
        // H = lse - E[a] = log Z - E[a - m]
        const float ent = gp - t.ss / t.r.zs;
        if (kl_out) kl_out[n] = kl;
        if (ent_out) ent_out[n] = ent;
        vals[n] = make_float2(kl, ent);
      }
    }
    par ^= 1;
  }
}

// acc[B,3] += {rows with mask = 1, sum kl, sum entropy} per sample; deterministic (one CTA
// per sample, fixed strided partials, fixed tree, fp64), accumulates across chunks.
static __global__ void __launch_bounds__(kSegThreads)
    divergence_reduce_kernel(const int32_t *sid, const uint8_t *mask, int64_t n_rows, const float2 *vals,
                             const unsigned long long *bounds, double *out) {
  __shared__ double sh[3][kSegThreads];
  __shared__ unsigned long long range_sh[2];
  const int32_t i = blockIdx.x;
  unsigned long long lo_u, hi_u;
  if (bounds) {
    lo_u = bounds[2 * (int64_t)i];
    hi_u = bounds[2 * (int64_t)i + 1];
  } else {
    sample_row_range(sid, n_rows, i, range_sh, lo_u, hi_u);
  }
  if (lo_u >= hi_u) return;
  const int64_t lo = (int64_t)lo_u, hi = (int64_t)hi_u;
  double cnt = 0.0, skl = 0.0, sen = 0.0;
  for (int64_t n = lo + threadIdx.x; n < hi; n += kSegThreads) {
    if (sid[n] != i || mask[n] == 0) continue;
    const float2 v = vals[n];
    cnt += 1.0;
    skl += (double)v.x;
    sen += (double)v.y;
  }
  sh[0][threadIdx.x] = cnt;
  sh[1][threadIdx.x] = skl;
  sh[2][threadIdx.x] = sen;
  __syncthreads();
  for (int off = kSegThreads / 2; off > 0; off >>= 1) {
    if (threadIdx.x < off)
      for (int j = 0; j < 3; ++j) sh[j][threadIdx.x] += sh[j][threadIdx.x + off];
    __syncthreads();
  }
  if (threadIdx.x == 0)
    for (int j = 0; j < 3; ++j) out[3 * (int64_t)i + j] += sh[j][0];
}

// Per-sample means: D_sup_i = sum kl / |U_i^sup| (Eq. 10, second row), m_sup_i = |U_i^sup| / H_i
// (Algorithm 1), mean entropy.  |U_i^sup| = 0: D_sup_i = +inf, which fopd_sample_freshness
// reads as "invalid for optimisation" (Algorithm 1), m_sup_i = 0.
static __global__ void __launch_bounds__(256)
    supervision_drift_kernel(const double *acc, const int32_t *H, int32_t B, float *d_sup, float *m_sup,
                             float *mean_entropy) {
  for (int32_t i = threadIdx.x; i < B; i += 256) {
    const double cnt = acc[3 * (int64_t)i];
    const int32_t h = H[i];
    const bool ok = cnt > 0.0;
    if (d_sup) d_sup[i] = ok ? (float)(fmax(acc[3 * (int64_t)i + 1], 0.0) / cnt) : __int_as_float(0x7f800000);
    if (m_sup) m_sup[i] = (ok && h > 0) ? (float)(cnt / (double)h) : 0.f;
    if (mean_entropy) mean_entropy[i] = ok ? (float)(acc[3 * (int64_t)i + 2] / cnt) : 0.f;
  }
}

// Buffer statistics of Eq. 14 and the refresh rule of Eq. 15 with its operators as printed
// (mean f <= kappa_f, mean m < kappa), at most one trigger per min_interval steps (Appendix B).
// decision[0]: bit 0 freshness, bit 1 rollout alignment, bit 2 supervision alignment,
// bit 3 = a condition holds but the interval has not passed; decision[1] = 1 if the buffer
// is to be refreshed now.
static __global__ void __launch_bounds__(256)
    refresh_decision_kernel(const float *f, const float *m_roll, const float *m_sup, int32_t B, float kappa_f,
                            float kappa_roll, float kappa_sup, int64_t steps_since_refresh, int64_t min_interval,
                            float *means, int32_t *decision) {
  __shared__ double sh[3][256];
  double a = 0.0, b = 0.0, c = 0.0;
  for (int32_t i = threadIdx.x; i < B; i += 256) {
    a += (double)f[i];
    b += (double)m_roll[i];
    c += (double)(m_sup ? m_sup[i] : m_roll[i]);
  }
  sh[0][threadIdx.x] = a;
  sh[1][threadIdx.x] = b;
  sh[2][threadIdx.x] = c;
  __syncthreads();
  for (int off = 128; off > 0; off >>= 1) {
    if (threadIdx.x < off)
      for (int j = 0; j < 3; ++j) sh[j][threadIdx.x] += sh[j][threadIdx.x + off];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const float fm = (float)(sh[0][0] / (double)B), mr = (float)(sh[1][0] / (double)B),
                ms = (float)(sh[2][0] / (double)B);
    if (means) {
      means[0] = fm;
      means[1] = mr;
      means[2] = ms;
    }
    int32_t bits = (fm <= kappa_f ? 1 : 0) | (mr < kappa_roll ? 2 : 0) | (ms < kappa_sup ? 4 : 0);
    const bool due = steps_since_refresh >= min_interval;
    if (bits && !due) bits |= 8;
    decision[0] = bits;
    decision[1] = (bits & 7) && due ? 1 : 0;
  }
}

}  // namespace fopd
