// Rows whose vocabulary is split over several holders (a tensor-parallel LM head):
// every holder sweeps its columns [v0, v0 + W) of each row into partial sums, the
// partial sums of all holders are merged into the row statistics of Sec. 4.1 /
// Eq. 10 / Eq. 12 (the exchange between holders is the caller's: [n_rows, 8] floats
// per holder), and every holder then writes the gradient of its own columns from
// the merged statistics.  The merged result is the whole-row result up to the order
// of the floating-point sums; the merge itself runs in a fixed order (part 0 first).
#pragma once

#include "stream_kernels.cuh"

namespace fopd {

constexpr int kPartialFloats = 8;  // FOPD_PART_* columns

// Partial sums of one shard.  c is the shard's view: logits point at column v0 of the full
// rows, c.vocab = W; tokens are ids in the full vocabulary.  Rows with mask = 0 are not read
// (zeros); sample ids and the token's range are judged at the merge, which sees all parts.
template <int DT, int kThreads>
__global__ void __launch_bounds__(kThreads, 1024 / kThreads)
    shard_stats_kernel(ChunkDev c, int64_t v0, float *partial) {
  using E = Elem<DT>;
  __shared__ RowAcc scratch[2][kThreads / 32];
  int par = 0;
  for (int64_t n = blockIdx.x; n < c.n_rows; n += gridDim.x) {
    float4 *out = reinterpret_cast<float4 *>(partial + n * kPartialFloats);
    if (c.mask[n] == 0) {
      if (threadIdx.x == 0) out[0] = out[1] = make_float4(0.f, 0.f, 0.f, 0.f);
      continue;
    }
    float sy = 0.f, ty = 0.f, has = 0.f;
    if (threadIdx.x == 0) {
      const int64_t y = (int64_t)c.tokens[n] - v0;
      if (y >= 0 && y < c.vocab) {
        sy = E::load1(c.student, n * c.stride + y);
        ty = E::load1(c.teacher, n * c.stride + y);
        has = 1.f;
      }
    }
    const char *srow = reinterpret_cast<const char *>(c.student) + n * c.stride * E::kBytes;
    const char *trow = reinterpret_cast<const char *>(c.teacher) + n * c.stride * E::kBytes;
    RowAcc acc = sweep_row_global<DT, kThreads>(srow, trow, c.vocab);
    acc = block_reduce<kThreads>(acc, scratch[par]);
    if (threadIdx.x == 0) {
      out[0] = make_float4(acc.ms, acc.zs, acc.as, acc.mt);
      out[1] = make_float4(acc.zt, sy, ty, has);
    }
    par ^= 1;
  }
}

// Merge of the parts of every row, one thread per row.  c carries the per-row side arrays and
// c.vocab = the full vocabulary (its logits pointers are not used).  A row whose token no part
// holds has a token outside the vocabulary: it is reported and treated as masked, like in the
// unsharded sweep.
static __global__ void __launch_bounds__(256)
    shard_merge_kernel(const float *partials, int32_t n_parts, ChunkDev c, int32_t B, float *lp_s, float *lp_t,
                       float *kl, float *ratio, float *row_ws, int32_t *status) {
  const int64_t n = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (n >= c.n_rows) return;
  if (!row_is_aligned(c, n, B, status, true)) {
    zero_row_outputs(n, lp_s, lp_t, kl, ratio, row_ws);
    return;
  }
  RowAcc r;
  r.init();
  float sy = 0.f, ty = 0.f, found = 0.f;
  for (int32_t k = 0; k < n_parts; ++k) {
    const float4 *p = reinterpret_cast<const float4 *>(partials + ((int64_t)k * c.n_rows + n) * kPartialFloats);
    const float4 a = p[0], b = p[1];
    RowAcc o;
    o.ms = a.x;
    o.zs = a.y;
    o.as = a.z;
    o.mt = a.w;
    o.zt = b.x;
    r.merge(o);
    if (b.w != 0.f) {
      sy = b.y;
      ty = b.z;
      found += 1.f;
    }
  }
  if (found != 1.f) {  // the parts do not tile the vocabulary the token was checked against
    if (status) atomicOr(status, FOPD_DEV_BAD_TOKEN);
    zero_row_outputs(n, lp_s, lp_t, kl, ratio, row_ws);
    return;
  }
  finish_row<FOPD_F32>(n, r, sy, ty, c.behav[n], FOPD_LOSS_FULL_KL, lp_s, lp_t, kl, ratio, row_ws);
}

// Gradient of one shard's columns from the merged row statistics.  c is the shard's view
// (as for shard_stats_kernel); v_total is the full vocabulary, against which tokens are judged.
template <int DT, int kThreads>
__global__ void __launch_bounds__(kThreads, 1024 / kThreads)
    shard_grad_kernel(ChunkDev c, int64_t v0, int64_t v_total, int32_t B, const float *coef, const float *row_ws,
                      float lambda, void *dlogits) {
  using E = Elem<DT>;
  for (int64_t n = blockIdx.x; n < c.n_rows; n += gridDim.x) {
    char *orow = reinterpret_cast<char *>(dlogits) + n * c.stride * E::kBytes;
    const int32_t sid = c.sid[n], y = c.tokens[n];
    const uint8_t m = c.mask[n];
    const float4 ws = reinterpret_cast<const float4 *>(row_ws)[n];
    float cf = (sid >= 0 && sid < B) ? coef[sid] : 0.f;
    if (m == 0 || y < 0 || y >= v_total) cf = 0.f;
    if (!(cf > 0.f)) {
      zero_fill_row<DT, kThreads>(orow, c.vocab);
      continue;
    }
    const int64_t yl = (int64_t)y - v0;
    const GradRow r = make_grad_row(ws, cf, lambda, (yl >= 0 && yl < c.vocab) ? (int32_t)yl : -1);
    grad_row_sweep<DT, kThreads>(reinterpret_cast<const char *>(c.student) + n * c.stride * E::kBytes,
                                 reinterpret_cast<const char *>(c.teacher) + n * c.stride * E::kBytes, orow, c.vocab,
                                 r);
  }
}

}  // namespace fopd
