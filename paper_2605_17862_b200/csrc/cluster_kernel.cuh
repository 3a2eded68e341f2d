// Fused loss forward + backward with the row resident on chip (sm_100a).
//
// A thread-block cluster owns one token row at a time.  Each CTA of the
// cluster stages its slice of the student and teacher rows in shared memory
// with bulk asynchronous copies (global -> shared, completion on mbarriers),
// runs the online max / sum-exp / KL sweep over it, and publishes its partial
// sums to every CTA of the cluster through distributed shared memory.  Once
// the cluster barrier has completed every CTA holds the row's normalisers and
// KL, and the gradient sweep reads the slice back from shared memory and
// streams dlogits out.  Student and teacher logits are read from HBM once and
// dlogits written once: 3 * V * e bytes per differentiated row.
//
// The rows of a cluster move through a three-stage software pipeline over three
// slice buffers per CTA:
//
//     step k:   reduction sweep of row k     (buffer k % 3), publish, barrier arrive
//               gradient sweep of row k - 1  (buffer (k - 1) % 3)
//               start the copies of row k + 2 into the buffer just freed
//               barrier wait, row constants of row k
//
// so the copies of a row are in flight for a whole step before they are
// needed, and the latency of the cluster exchange of row k is covered by the
// gradient sweep of row k - 1.  A small kernel run first writes each row's
// weight coef_i (0 for rows that are not differentiated), which lets the
// pipeline look rows ahead with independent loads.
//
// Waits on the copy barriers are bounded; if one ever runs out the CTA records
// FOPD_DEV_TIMEOUT in the status word and keeps taking part in the cluster
// barriers (so that no peer is left waiting) until the kernel ends.
#pragma once

#include "stream_kernels.cuh"

namespace fopd {

constexpr int kClusterThreads = 1024;
constexpr int kMaxClusterSize = 16;
constexpr int kSliceBufs = 3;
constexpr int kMaxChunks = 8;                // copy chunks (and mbarriers) per slice buffer
constexpr uint32_t kSpinLimit = 1u << 22;    // polls of one mbarrier before giving up

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t cluster_nctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: false if the phase did not complete within kSpinLimit polls.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
  for (uint32_t i = 0; i < kSpinLimit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if (i > 64) __nanosleep(64);
  }
  return false;
}
__device__ __forceinline__ void bulk_load(uint32_t dst_smem, const void *src, uint32_t bytes, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst_smem),
      "l"(src), "r"(bytes), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void cluster_arrive() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_wait() {
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_smem, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_smem), "r"(rank));
  return r;
}
__device__ __forceinline__ void st_cluster_f32(uint32_t addr, float v) {
  asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}

// Cheaper merge for reductions: agree on the maxima first, rescale once, then add.
__device__ __forceinline__ RowAcc warp_reduce_two_step(RowAcc a) {
  float Ms = a.ms, Mt = a.mt;
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    Ms = fmaxf(Ms, __shfl_xor_sync(0xffffffffu, Ms, off));
    Mt = fmaxf(Mt, __shfl_xor_sync(0xffffffffu, Mt, off));
  }
  const float rs = ex2((a.ms - Ms) * kLog2e), rt = ex2((a.mt - Mt) * kLog2e);
  a.zs *= rs;
  a.as *= rs;
  a.zt *= rt;
  a.ms = Ms;
  a.mt = Mt;
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    a.zs += __shfl_xor_sync(0xffffffffu, a.zs, off);
    a.as += __shfl_xor_sync(0xffffffffu, a.as, off);
    a.zt += __shfl_xor_sync(0xffffffffu, a.zt, off);
  }
  return a;
}

// Weight of every row of a chunk: coef of its sample if the row is differentiated
// (aligned, ids in range, coef > 0), else 0.  Reports bad ids in the status word.
static __global__ void __launch_bounds__(256)
    row_coef_kernel(ChunkDev c, int32_t B, const float *coef, int32_t *status, float *row_cf) {
  const int64_t n = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (n >= c.n_rows) return;
  float cf = 0.f;
  if (row_is_aligned(c, n, B, status, true)) cf = coef[c.sid[n]];
  row_cf[n] = cf > 0.f ? cf : 0.f;
}

struct ClusterShared {
  unsigned long long load_bar[kSliceBufs][kMaxChunks];  // one mbarrier per copy chunk (S and T land on it)
  RowAcc partial[2][kMaxClusterSize];        // [row parity][source CTA rank], written by peers through DSMEM
  float token_logit[2];                      // [row parity] S[n, y_n], written by the CTA whose slice holds it
  RowAcc warp_scratch[kClusterThreads / 32];
  GradRow grad_row[2];                       // [row parity] constants of the gradient sweep, set by thread 0
  int failed;
};

struct FusedArgs {
  ChunkDev c;
  float lambda;
  void *dlogits;
  const float *row_cf;  // [n_rows] from row_coef_kernel
  float *row_ws;        // [n_rows,4] out: {lse_s, lse_t, kl, d}; zeros for rows not differentiated
  int32_t *status;
  int slice_vecs;       // 16-byte vectors of a row per CTA (the last CTAs' slices may be shorter or empty)
};

template <int DT>
__global__ void __launch_bounds__(kClusterThreads, 1) fused_cluster_kernel(FusedArgs a) {
  using E = Elem<DT>;
  constexpr int P = E::kPerVec;
  constexpr int kThreads = kClusterThreads;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  ClusterShared &sh = *reinterpret_cast<ClusterShared *>(smem_raw);
  const uint32_t data_off = (sizeof(ClusterShared) + 127u) & ~127u;
  const uint32_t slice_bytes = (uint32_t)a.slice_vecs * 16u;
  const uint32_t data_base = smem_u32(smem_raw) + data_off;   // buffer k: S slice at +2k*slice_bytes, T after it

  const uint32_t rank = cluster_ctarank(), csize = cluster_nctarank();
  const int64_t n_clusters = gridDim.x / csize, cluster_id = blockIdx.x / csize;
  const ChunkDev &c = a.c;
  const int64_t V = c.vocab, nvec = V / P;
  const int tid = threadIdx.x;

  // This CTA's slice of every row, in vectors.
  const int64_t v_lo = (int64_t)rank * a.slice_vecs;
  const int my_vecs = (int)max((int64_t)0, min((int64_t)a.slice_vecs, nvec - v_lo));
  const int n_chunks = (my_vecs + kThreads - 1) / kThreads;
  const bool owns_tail = (rank == csize - 1);
  const int64_t tail_idx = nvec * P + tid;  // scalar tail element handled by the last CTA
  const int64_t row_bytes = c.stride * E::kBytes;

  if (tid == 0) {
    for (int b = 0; b < kSliceBufs; ++b)
      for (int k = 0; k < kMaxChunks; ++k) mbar_init(smem_u32(&sh.load_bar[b][k]), 1);
    sh.failed = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  cluster_arrive();
  cluster_wait();

  // Thread 0 starts the copies of row n's slice into buffer `buf`: one bulk copy per tensor per chunk.
  auto issue_row = [&](int64_t n, uint32_t buf) {
    const char *srow = reinterpret_cast<const char *>(c.student) + n * row_bytes + v_lo * 16;
    const char *trow = reinterpret_cast<const char *>(c.teacher) + n * row_bytes + v_lo * 16;
    const uint32_t s_base = data_base + buf * 2u * slice_bytes, t_base = s_base + slice_bytes;
    for (int k = 0; k < n_chunks; ++k) {
      const int v0 = k * kThreads;
      const uint32_t bytes = (uint32_t)min(kThreads, my_vecs - v0) * 16u;
      const uint32_t bar = smem_u32(&sh.load_bar[buf][k]);
      mbar_expect_tx(bar, 2u * bytes);
      bulk_load(s_base + (uint32_t)v0 * 16u, srow + (int64_t)v0 * 16, bytes, bar);
      bulk_load(t_base + (uint32_t)v0 * 16u, trow + (int64_t)v0 * 16, bytes, bar);
    }
  };

  // ---- scan over this cluster's rows, row weights fetched three rows ahead
  auto load_cf = [&](int64_t n) { return n < c.n_rows ? __ldg(a.row_cf + n) : 0.f; };
  int64_t scan_n = cluster_id;
  float cf0 = load_cf(scan_n), cf1 = load_cf(scan_n + n_clusters), cf2 = load_cf(scan_n + 2 * n_clusters);
  // Next differentiated row (or -1 when the rows are exhausted); rows passed on the way are
  // not differentiated and get their zeros here.
  auto next_row = [&](float &cf_out) -> int64_t {
    while (scan_n < c.n_rows) {
      const int64_t n = scan_n;
      const float cf = cf0;
      cf0 = cf1;
      cf1 = cf2;
      cf2 = load_cf(scan_n + 3 * n_clusters);
      scan_n += n_clusters;
      if (cf > 0.f) {
        cf_out = cf;
        return n;
      }
      char *orow = reinterpret_cast<char *>(a.dlogits) + n * row_bytes;
      uint4 *o4 = reinterpret_cast<uint4 *>(orow) + v_lo;
      const uint4 z = make_uint4(0u, 0u, 0u, 0u);
      for (int i = tid; i < my_vecs; i += kThreads) st_stream(o4 + i, z);
      if (owns_tail && tail_idx < V) E::store1(orow, tail_idx, 0.f);
      if (rank == 0 && tid == 0) reinterpret_cast<float4 *>(a.row_ws)[n] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    cf_out = 0.f;
    return -1;
  };

  // Rows in the pipeline: row_g awaits its gradient sweep, row_r its reduction sweep (copies
  // issued), row_l has its copies issued.  k counts the differentiated rows: row_r is number k.
  float cf_r = 0.f, cf_l = 0.f;
  int64_t row_g = -1;
  int64_t row_r = next_row(cf_r);
  if (row_r >= 0 && tid == 0) issue_row(row_r, 0);
  int64_t row_l = row_r >= 0 ? next_row(cf_l) : -1;
  if (row_l >= 0 && tid == 0) issue_row(row_l, 1);

  for (uint32_t k = 0; row_r >= 0 || row_g >= 0; ++k) {
    // side inputs of row k that warp 0 needs after the sweep: fetched now, used late
    int32_t y = 0;
    float b = 0.f;
    if (row_r >= 0 && tid < 32) {
      y = c.tokens[row_r];
      b = c.behav[row_r];
    }
    // ---- reduction sweep of row k
    if (row_r >= 0) {
      const uint32_t buf = k % kSliceBufs, parity = (k / kSliceBufs) & 1u, slot = k & 1u;
      const uint32_t s_base = data_base + buf * 2u * slice_bytes, t_base = s_base + slice_bytes;
      const char *srow = reinterpret_cast<const char *>(c.student) + row_r * row_bytes;
      const char *trow = reinterpret_cast<const char *>(c.teacher) + row_r * row_bytes;

      RowAcc acc;
      acc.init();
      bool ok = true;
      for (int kc = 0; kc < n_chunks; ++kc) {
        ok = mbar_wait_bounded(smem_u32(&sh.load_bar[buf][kc]), parity) && ok;
        const int i = kc * kThreads + tid;
        if (i < my_vecs) {
          float s[P], t[P];
          E::unpack(lds128(s_base + (uint32_t)i * 16u), s);
          E::unpack(lds128(t_base + (uint32_t)i * 16u), t);
          acc.add<P>(s, t);
        }
      }
      if (!ok) sh.failed = 1;
      if (owns_tail && tail_idx < V) acc.add1(E::load1(srow, tail_idx), E::load1(trow, tail_idx));

      // CTA partial (and the stored token's logit) published to every CTA through DSMEM
      acc = warp_reduce_two_step(acc);
      if ((tid & 31) == 0) sh.warp_scratch[tid >> 5] = acc;
      __syncthreads();  // also publishes grad_row of row k - 1 to the gradient sweep below
      if (tid < 32) {
        RowAcc r = sh.warp_scratch[tid];
        r = warp_reduce_two_step(r);
        // which CTA holds S[n, y]: the slice that contains its vector, or the last CTA for the scalar tail
        const int64_t yv = y / P;
        const bool in_body = yv < nvec;
        const bool mine = in_body ? (yv >= v_lo && yv < v_lo + my_vecs) : owns_tail;
        float sy = 0.f;
        if (mine) {
          if (in_body) {
            const uint32_t addr = s_base + (uint32_t)((int64_t)y - v_lo * P) * E::kBytes;
            if (DT == FOPD_BF16) {
              unsigned short h;
              asm volatile("ld.shared.u16 %0, [%1];" : "=h"(h) : "r"(addr));
              sy = __uint_as_float(((uint32_t)h) << 16);
            } else {
              asm volatile("ld.shared.f32 %0, [%1];" : "=f"(sy) : "r"(addr));
            }
          } else {
            sy = E::load1(srow, y);
          }
        }
        if (tid < (int)csize) {
          const uint32_t dst = map_to_cta(smem_u32(&sh.partial[slot][rank]), (uint32_t)tid);
          st_cluster_f32(dst + 0, r.ms);
          st_cluster_f32(dst + 4, r.zs);
          st_cluster_f32(dst + 8, r.as);
          st_cluster_f32(dst + 12, r.mt);
          st_cluster_f32(dst + 16, r.zt);
          if (mine) st_cluster_f32(map_to_cta(smem_u32(&sh.token_logit[slot]), (uint32_t)tid), sy);
        }
      }
      cluster_arrive();
    } else {
      __syncthreads();  // publishes grad_row of the last row
    }

    // ---- gradient sweep of row k - 1 from its resident slice, streamed out
    if (row_g >= 0) {
      const uint32_t buf = (k + kSliceBufs - 1) % kSliceBufs;
      const uint32_t s_base = data_base + buf * 2u * slice_bytes, t_base = s_base + slice_bytes;
      const GradRow gr = sh.grad_row[(k + 1) & 1u];
      char *orow = reinterpret_cast<char *>(a.dlogits) + row_g * row_bytes;
      uint4 *o4 = reinterpret_cast<uint4 *>(orow) + v_lo;
      for (int i = tid; i < my_vecs; i += kThreads) {
        const uint4 sv = lds128(s_base + (uint32_t)i * 16u), tv = lds128(t_base + (uint32_t)i * 16u);
        st_stream(o4 + i, grad_vec<DT>(sv, tv, gr, (v_lo + i) * P));
      }
      if (owns_tail && tail_idx < V) {
        const char *srow = reinterpret_cast<const char *>(c.student) + row_g * row_bytes;
        const char *trow = reinterpret_cast<const char *>(c.teacher) + row_g * row_bytes;
        const float s = E::load1(srow, tail_idx), t = E::load1(trow, tail_idx);
        float o = ex2(fmaf(s, kLog2e, gr.e0)) * ((s - t) - gr.K);
        if (tail_idx == gr.y) o += gr.cg;
        E::store1(orow, tail_idx, o);
      }
    }
    __syncthreads();  // the buffer of row k - 1 is free

    // ---- look ahead: row k + 2 goes into the buffer just freed ((k + 2) % 3 == (k - 1) % 3)
    float cf_n = 0.f;
    const int64_t row_n = row_l >= 0 ? next_row(cf_n) : -1;
    if (row_n >= 0 && tid == 0) issue_row(row_n, (k + 2) % kSliceBufs);

    // ---- finish the exchange of row k: row constants, identical in every CTA
    if (row_r >= 0) {
      cluster_wait();
      if (tid == 0) {
        const uint32_t slot = k & 1u;
        RowAcc r = sh.partial[slot][0];
        for (uint32_t j = 1; j < csize; ++j) r.merge(sh.partial[slot][j]);
        const float ls = r.ms + logf(r.zs), lt = r.mt + logf(r.zt);
        const float kl = r.as / r.zs - (ls - lt);
        const float d = (sh.token_logit[slot] - ls) - b;
        sh.grad_row[slot] = make_grad_row(make_float4(ls, lt, kl, d), cf_r, a.lambda, y);
        if (rank == 0) reinterpret_cast<float4 *>(a.row_ws)[row_r] = make_float4(ls, lt, kl, d);
      }
    }
    row_g = row_r;
    row_r = row_l;
    cf_r = cf_l;
    row_l = row_n;
    cf_l = cf_n;
  }

  if (tid == 0 && sh.failed && a.status) atomicOr(a.status, FOPD_DEV_TIMEOUT);
  // No CTA may exit while a peer can still write into its shared memory.
  cluster_arrive();
  cluster_wait();
}

}  // namespace fopd
