// Fused loss forward + backward with the row resident on chip (sm_100a).
//
// A thread-block cluster owns one token row at a time.  Each CTA of the
// cluster stages its slice of the student and teacher rows in shared memory
// with bulk asynchronous copies (global -> shared, completion on mbarriers),
// runs the online max / sum-exp / KL sweep over it as the chunks land, and
// publishes its partial sums to every CTA of the cluster through distributed
// shared memory.  After one cluster barrier every CTA holds the row's
// normalisers and KL, and the gradient sweep reads the slice back from shared
// memory and streams dlogits out.  Student and teacher logits are read from
// HBM once and dlogits written once: 3 * V * e bytes per differentiated row.
//
// Waits on the copy barriers are bounded; if one ever runs out the CTA records
// FOPD_DEV_TIMEOUT in the status word and keeps taking part in the cluster
// barriers (so that no peer is left waiting) until the kernel ends.
#pragma once

#include "stream_kernels.cuh"

namespace fopd {

constexpr int kClusterThreads = 512;
constexpr int kMaxClusterSize = 16;
constexpr int kMaxChunks = 32;               // copy chunks (and mbarriers) per slice
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

struct ClusterShared {
  unsigned long long load_bar[kMaxChunks];   // one mbarrier per copy chunk (S and T chunk both land on it)
  RowAcc partial[2][kMaxClusterSize];        // [row parity][source CTA rank], written by peers through DSMEM
  RowAcc warp_scratch[kClusterThreads / 32];
  GradRow grad_row;                          // per-row constants of the gradient sweep, broadcast by thread 0
  float row_stats[4];
  int failed;
};

struct FusedArgs {
  ChunkDev c;
  int32_t B;
  const float *coef;
  float lambda;
  void *dlogits;
  float *row_ws;       // [n_rows,4] out: {lse_s, lse_t, kl, d}; zeros for rows not differentiated
  int32_t *status;
  int slice_vecs;      // 16-byte vectors of a row per CTA (the last CTA's slice may be shorter)
  int chunk_vecs;      // vectors per copy chunk (= kClusterThreads)
};

template <int DT>
__global__ void __launch_bounds__(kClusterThreads, 2) fused_cluster_kernel(FusedArgs a) {
  using E = Elem<DT>;
  constexpr int P = E::kPerVec;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  ClusterShared &sh = *reinterpret_cast<ClusterShared *>(smem_raw);
  const uint32_t data_off = (sizeof(ClusterShared) + 127u) & ~127u;
  const uint32_t slice_bytes = (uint32_t)a.slice_vecs * 16u;
  const uint32_t s_base = smem_u32(smem_raw) + data_off;
  const uint32_t t_base = s_base + slice_bytes;

  const uint32_t rank = cluster_ctarank(), csize = cluster_nctarank();
  const int64_t n_clusters = gridDim.x / csize, cluster_id = blockIdx.x / csize;
  const ChunkDev &c = a.c;
  const int64_t V = c.vocab, nvec = V / P;
  const int tid = threadIdx.x;

  // This CTA's slice of every row, in vectors.
  const int64_t v_lo = (int64_t)rank * a.slice_vecs;
  const int my_vecs = (int)max((int64_t)0, min((int64_t)a.slice_vecs, nvec - v_lo));
  const int n_chunks = (my_vecs + a.chunk_vecs - 1) / a.chunk_vecs;
  const bool owns_tail = (rank == csize - 1);
  const int64_t tail_idx = nvec * P + tid;  // scalar tail element handled by the last CTA

  if (tid == 0) {
    for (int k = 0; k < kMaxChunks; ++k) mbar_init(smem_u32(&sh.load_bar[k]), 1);
    sh.failed = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  cluster_arrive();
  cluster_wait();

  uint32_t phase = 0;  // parity of the copy barriers and of the partial slots; flips per differentiated row
  for (int64_t n = cluster_id; n < c.n_rows; n += n_clusters) {
    char *orow = reinterpret_cast<char *>(a.dlogits) + n * c.stride * E::kBytes;
    uint4 *o4 = reinterpret_cast<uint4 *>(orow) + v_lo;
    float cf = 0.f;
    if (row_is_aligned(c, n, a.B, a.status, tid == 0 && rank == 0)) cf = a.coef[c.sid[n]];
    if (!(cf > 0.f)) {  // every CTA of the cluster takes this branch together
      const uint4 z = make_uint4(0u, 0u, 0u, 0u);
      for (int i = tid; i < my_vecs; i += kClusterThreads) st_stream(o4 + i, z);
      if (owns_tail && tail_idx < V) E::store1(orow, tail_idx, 0.f);
      if (rank == 0 && tid == 0) reinterpret_cast<float4 *>(a.row_ws)[n] = make_float4(0.f, 0.f, 0.f, 0.f);
      continue;
    }
    const char *srow = reinterpret_cast<const char *>(c.student) + n * c.stride * E::kBytes;
    const char *trow = reinterpret_cast<const char *>(c.teacher) + n * c.stride * E::kBytes;

    // ---- stage the slice: one bulk copy per tensor per chunk
    if (tid == 0) {
      for (int k = 0; k < n_chunks; ++k) {
        const int v0 = k * a.chunk_vecs;
        const uint32_t bytes = (uint32_t)min(a.chunk_vecs, my_vecs - v0) * 16u;
        const uint32_t bar = smem_u32(&sh.load_bar[k]);
        mbar_expect_tx(bar, 2u * bytes);
        bulk_load(s_base + (uint32_t)v0 * 16u, srow + (v_lo + v0) * 16, bytes, bar);
        bulk_load(t_base + (uint32_t)v0 * 16u, trow + (v_lo + v0) * 16, bytes, bar);
      }
    }

    // ---- sweep 1: online max / sum-exp / KL accumulators over the slice as chunks land
    RowAcc acc;
    acc.init();
    bool ok = true;
    for (int k = 0; k < n_chunks; ++k) {
      ok = mbar_wait_bounded(smem_u32(&sh.load_bar[k]), phase) && ok;
      const int i = k * a.chunk_vecs + tid;
      if (i < my_vecs) {
        float s[P], t[P];
        E::unpack(lds128(s_base + (uint32_t)i * 16u), s);
        E::unpack(lds128(t_base + (uint32_t)i * 16u), t);
        acc.add<P>(s, t);
      }
    }
    if (!ok) sh.failed = 1;
    if (owns_tail && tail_idx < V) acc.add1(E::load1(srow, tail_idx), E::load1(trow, tail_idx));

    // ---- CTA partial, published to every CTA of the cluster through DSMEM
    acc = warp_reduce_two_step(acc);
    if ((tid & 31) == 0) sh.warp_scratch[tid >> 5] = acc;
    __syncthreads();
    if (tid < 32) {
      RowAcc r;
      r.init();
      if (tid < kClusterThreads / 32) r = sh.warp_scratch[tid];
      r = warp_reduce_two_step(r);
      if (tid < (int)csize) {
        const uint32_t dst = map_to_cta(smem_u32(&sh.partial[phase][rank]), (uint32_t)tid);
        st_cluster_f32(dst + 0, r.ms);
        st_cluster_f32(dst + 4, r.zs);
        st_cluster_f32(dst + 8, r.as);
        st_cluster_f32(dst + 12, r.mt);
        st_cluster_f32(dst + 16, r.zt);
      }
    }
    cluster_arrive();
    cluster_wait();

    // ---- row scalars (identical in every CTA: same partials, same order)
    if (tid == 0) {
      RowAcc r = sh.partial[phase][0];
      for (uint32_t j = 1; j < csize; ++j) r.merge(sh.partial[phase][j]);
      const float ls = r.ms + logf(r.zs), lt = r.mt + logf(r.zt);
      const float kl = r.as / r.zs - (ls - lt);
      const int32_t y = c.tokens[n];
      const float d = (E::load1(c.student, n * c.stride + y) - ls) - c.behav[n];
      sh.grad_row = make_grad_row(make_float4(ls, lt, kl, d), cf, a.lambda, y);
      if (rank == 0) reinterpret_cast<float4 *>(a.row_ws)[n] = make_float4(ls, lt, kl, d);
    }
    __syncthreads();
    const GradRow gr = sh.grad_row;

    // ---- sweep 2: gradient from the resident slice, streamed out
    for (int i = tid; i < my_vecs; i += kClusterThreads) {
      const uint4 sv = lds128(s_base + (uint32_t)i * 16u), tv = lds128(t_base + (uint32_t)i * 16u);
      st_stream(o4 + i, grad_vec<DT>(sv, tv, gr, (v_lo + i) * P));
    }
    if (owns_tail && tail_idx < V) {
      const float s = E::load1(srow, tail_idx), t = E::load1(trow, tail_idx);
      float o = ex2(fmaf(s, kLog2e, gr.e0)) * ((s - t) - gr.K);
      if (tail_idx == gr.y) o += gr.cg;
      E::store1(orow, tail_idx, o);
    }
    phase ^= 1u;
    __syncthreads();  // the slice is free for the next row's copies
  }

  if (tid == 0 && sh.failed && a.status) atomicOr(a.status, FOPD_DEV_TIMEOUT);
  // No CTA may exit while a peer can still write into its shared memory.
  cluster_arrive();
  cluster_wait();
}

}  // namespace fopd
