// Fused loss forward + backward with the row resident on chip (sm_100a).
//
// A thread-block cluster owns one token row at a time.  Each CTA of the
// cluster stages its slice of the student and teacher rows in shared memory
// with bulk asynchronous copies (global -> shared, completion on an mbarrier),
// runs the online max / sum-exp / KL sweep over it, and sends its partial sums
// to every CTA of the cluster through distributed shared memory.  Once all
// partials have landed every CTA holds the row's normalisers and KL, and the
// gradient sweep reads the slice back from shared memory and streams dlogits
// out.  Student and teacher logits are read from HBM once and dlogits written
// once: 3 * V * e bytes per differentiated row.
//
// Warp 0 of each CTA is a control warp, the other warps compute.  The rows of
// a cluster move through a software pipeline over three slice buffers per CTA:
//
//   compute warps, step k:  reduction sweep of row k     (buffer k % 3)
//                           gradient sweep of row k - 1  (buffer (k - 1) % 3)
//   control warp,  step k:  merge the warps' partials of row k, send them to
//                           the cluster; start the copies of row k + 2 into
//                           the buffer of row k - 1 once its gradient sweep is
//                           done; when all CTAs' partials of row k are here,
//                           form the row constants for its gradient sweep
//
// so the copies of a row are in flight for a whole step before they are
// needed and the cluster exchange of row k is covered by the gradient sweep of
// row k - 1.  All hand-offs inside a CTA and between CTAs go through mbarriers
// (no CTA-wide or cluster-wide barrier inside the loop).  A small kernel run
// first writes each row's weight coef_i (0 for rows that are not
// differentiated), which lets the pipeline look rows ahead with independent
// loads.
//
// Every mbarrier wait is bounded; if one runs out the thread records
// FOPD_DEV_TIMEOUT in the status word, skips its remaining waits and runs to
// the end of the kernel (the results of that call are void).
#pragma once

#include "stream_kernels.cuh"

namespace fopd {

// Block sizes the kernel is built for.  Warp 0 is the control warp, the others compute; the
// launcher picks the size whose compute threads share a slice most evenly (a thread sweeps
// only a few vectors per row, so an uneven split idles a large part of the block).
#define FOPD_CLUSTER_THREAD_CHOICES(X) X(512) X(640) X(768) X(896) X(1024)
constexpr int kMaxClusterSize = 16;
constexpr int kSliceBufs = 3;
constexpr long long kWaitCycles = 200000000;  // SM cycles one mbarrier wait may take before giving up (~0.1 s)

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
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Arrival that orders nothing: for "done reading this buffer" signals, issued after the
// instructions that consumed the data read.
__device__ __forceinline__ void mbar_arrive_relaxed(uint32_t bar) {
  asm volatile("mbarrier.arrive.relaxed.cta.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Stores into another CTA's shared memory that also credit their bytes to an mbarrier of
// that CTA: the receiver's wait on the barrier covers the data, the sender needs no fence.
__device__ __forceinline__ void st_async_v4(uint32_t cluster_addr, float a, float b, float c, float d,
                                            uint32_t cluster_bar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.f32 [%0], {%1, %2, %3, %4}, [%5];" ::"r"(
                   cluster_addr),
               "f"(a), "f"(b), "f"(c), "f"(d), "r"(cluster_bar)
               : "memory");
}
__device__ __forceinline__ void st_async_f32(uint32_t cluster_addr, float a, uint32_t cluster_bar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.f32 [%0], %1, [%2];" ::"r"(cluster_addr),
               "f"(a), "r"(cluster_bar)
               : "memory");
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
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded waits: false if the phase did not complete within kWaitCycles.  try_wait itself
// parks the thread for a while, so the loop is kept to the poll and a branch; the clock is
// read once per kPollsPerClock polls.
constexpr int kPollsPerClock = 256;
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  do {
    for (int i = 0; i < kPollsPerClock; ++i)
      if (mbar_try_wait(bar, parity)) return true;
  } while (clock64() - t0 <= kWaitCycles);
  return false;
}
__device__ __forceinline__ bool mbar_wait_cluster_bounded(uint32_t bar, uint32_t parity) {
  if (mbar_try_wait_cluster(bar, parity)) return true;
  const long long t0 = clock64();
  do {
    for (int i = 0; i < kPollsPerClock; ++i)
      if (mbar_try_wait_cluster(bar, parity)) return true;
  } while (clock64() - t0 <= kWaitCycles);
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
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
// One logit from a staged slice.
template <int DT>
__device__ __forceinline__ float lds_logit(uint32_t addr) {
  float x;
  if (DT == FOPD_BF16) {
    unsigned short h;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(h) : "r"(addr));
    x = __uint_as_float(((uint32_t)h) << 16);
  } else {
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(x) : "r"(addr));
  }
  return x;
}
__device__ __forceinline__ float warp_max(float x) {
  float r;
  asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(x));
  return r;
}

// Warp-wide merge of per-lane accumulators: agree on the maxima first (one redux each),
// rescale once, then add.  The three sums travel in 10 shuffles instead of 15: in the
// first exchange each lane hands one of (zs, as) to its neighbour and keeps the other.
// Student and teacher sums are combined in the same order, so equal inputs give equal bits.
__device__ __forceinline__ RowAcc warp_reduce_two_step(RowAcc a) {
  const float Ms = warp_max(a.ms), Mt = warp_max(a.mt);
  const float rs = ex2((a.ms - Ms) * kLog2e), rt = ex2((a.mt - Mt) * kLog2e);
  const float zs = a.zs * rs, as = a.as * rs;
  float zt = a.zt * rt;
  const bool odd = threadIdx.x & 1;
  const float give = odd ? zs : as, keep = odd ? as : zs;  // even lanes collect zs, odd lanes as
  float za = keep + __shfl_xor_sync(0xffffffffu, give, 1);
  zt += __shfl_xor_sync(0xffffffffu, zt, 1);
#pragma unroll
  for (int off = 2; off < 32; off <<= 1) {
    za += __shfl_xor_sync(0xffffffffu, za, off);
    zt += __shfl_xor_sync(0xffffffffu, zt, off);
  }
  const float other = __shfl_xor_sync(0xffffffffu, za, 1);
  a.zs = odd ? other : za;
  a.as = odd ? za : other;
  a.zt = zt;
  a.ms = Ms;
  a.mt = Mt;
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
  unsigned long long load_bar[kSliceBufs];   // copies of a slice landed (1 arrival + bytes)
  unsigned long long free_bar[kSliceBufs];   // gradient sweep of the slice done (one arrival per compute warp)
  unsigned long long red_bar[2];             // [row parity] warp partials written (one arrival per compute warp)
  unsigned long long grad_bar[2];            // [row parity] grad_row ready (1 arrival)
  unsigned long long xchg_bar[2];            // [row parity] partials of all CTAs here (1 arrival + bytes)
  float4 partial4[2][kMaxClusterSize];       // [row parity][source CTA rank] {ms, zs, as, mt}, written by peers
  float partial_zt[2][kMaxClusterSize];      // [row parity][source CTA rank] zt
  float token_logit[2];                      // [row parity] S[n, y_n], written by the CTA whose slice holds it
  RowAcc warp_scratch[2][32];                // [row parity][compute warp]
  GradRow grad_row[2];                       // [row parity] constants of the gradient sweep
  long long row_after_next[2];               // [row parity] row k + 2 of this cluster (or -1), found by the control warp
  int2 token_patch[2];                       // [row parity] {compute thread that stores the token's vector or -1,
                                             //               byte offset of the token's logit in the slice}
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


template <int DT, int kThreads>
__global__ void __launch_bounds__(kThreads, 1) fused_cluster_kernel(FusedArgs a) {
  using E = Elem<DT>;
  constexpr int P = E::kPerVec;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  ClusterShared &sh = *reinterpret_cast<ClusterShared *>(smem_raw);
  const uint32_t data_off = (sizeof(ClusterShared) + 127u) & ~127u;
  const uint32_t slice_bytes = (uint32_t)a.slice_vecs * 16u;
  const uint32_t data_base = smem_u32(smem_raw) + data_off;   // buffer k: S slice at +2k*slice_bytes, T after it

  const uint32_t rank = cluster_ctarank(), csize = cluster_nctarank();
  const int64_t n_clusters = gridDim.x / csize, cluster_id = blockIdx.x / csize;
  const ChunkDev &c = a.c;
  const int64_t V = c.vocab, nvec = V / P;
  const int tid = threadIdx.x, lane = tid & 31;
  const bool control = tid < 32;
  const int ctid = tid - 32;   // index among the compute threads (negative in the control warp)
  constexpr int n_compute = kThreads - 32, n_compute_warps = n_compute / 32;

  // This CTA's slice of every row, in vectors.
  const int64_t v_lo = (int64_t)rank * a.slice_vecs;
  const int my_vecs = (int)max((int64_t)0, min((int64_t)a.slice_vecs, nvec - v_lo));
  const bool owns_tail = (rank == csize - 1);
  const int64_t tail_idx = nvec * P + ctid;  // scalar tail element handled by the last CTA's compute threads
  const bool has_tail = owns_tail && !control && tail_idx < V;
  const int64_t row_bytes = c.stride * E::kBytes;

  if (tid == 0) {
    for (int b = 0; b < kSliceBufs; ++b) {
      mbar_init(smem_u32(&sh.load_bar[b]), 1);
      mbar_init(smem_u32(&sh.free_bar[b]), n_compute_warps);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&sh.red_bar[b]), n_compute_warps);
      mbar_init(smem_u32(&sh.grad_bar[b]), 1);
      mbar_init(smem_u32(&sh.xchg_bar[b]), 1);
    }
    sh.failed = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  cluster_arrive();
  cluster_wait();

  // One thread starts the copies of row n's slice into buffer `buf`: one bulk copy per tensor.
  auto issue_row = [&](int64_t n, uint32_t buf) {
    if (my_vecs == 0) return;
    const char *srow = reinterpret_cast<const char *>(c.student) + n * row_bytes + v_lo * 16;
    const char *trow = reinterpret_cast<const char *>(c.teacher) + n * row_bytes + v_lo * 16;
    const uint32_t s_base = data_base + buf * 2u * slice_bytes, t_base = s_base + slice_bytes;
    const uint32_t bytes = (uint32_t)my_vecs * 16u, bar = smem_u32(&sh.load_bar[buf]);
    mbar_expect_tx(bar, 2u * bytes);
    bulk_load(s_base, srow, bytes, bar);
    bulk_load(t_base, trow, bytes, bar);
  };
  // After one wait has run out the rest are skipped: the results are void anyway and the
  // kernel must end soon.
  bool ok = true;
  auto wait_on = [&](unsigned long long *bar, uint32_t parity) {
    if (ok) ok = mbar_wait_bounded(smem_u32(bar), parity);
  };

  // This CTA's part of a row that is not differentiated: zeros (compute threads only).
  auto zero_row = [&](int64_t n) {
    char *orow = reinterpret_cast<char *>(a.dlogits) + n * row_bytes;
    uint4 *o4 = reinterpret_cast<uint4 *>(orow) + v_lo;
    const uint4 z = make_uint4(0u, 0u, 0u, 0u);
    if (!control)
      for (int i = ctid; i < my_vecs; i += n_compute) st_stream(o4 + i, z);
    if (has_tail) E::store1(orow, tail_idx, 0.f);
  };

  // ---- scan over this cluster's rows, row weights fetched three rows ahead.  Every thread
  // scans up to the first two differentiated rows; from then on only the control warp does.
  auto load_cf = [&](int64_t n) { return n < c.n_rows ? __ldg(a.row_cf + n) : 0.f; };
  int64_t scan_n = cluster_id;
  float cf0 = load_cf(scan_n), cf1 = load_cf(scan_n + n_clusters), cf2 = load_cf(scan_n + 2 * n_clusters);
  // Next differentiated row (or -1 when the rows are exhausted).  Rows passed on the way are
  // not differentiated: they get their zeros here if compute threads take part in the call,
  // else from the compute warps when they learn of the next row.
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
      zero_row(n);
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
    const uint32_t slot = k & 1u, par2 = (k >> 1) & 1u;
    const uint32_t buf_r = k % kSliceBufs, buf_g = (k + kSliceBufs - 1) % kSliceBufs;
    float cf_n = 0.f;
    int64_t row_n = -1;
    if (control) {
      // =================================================== control warp
      int32_t y = 0;
      float b = 0.f, sy = 0.f;
      if (row_r >= 0) {
        y = c.tokens[row_r];   // used after the waits below
        b = c.behav[row_r];
        sy = E::load1(reinterpret_cast<const char *>(c.student) + row_r * row_bytes, y);
        // CTA partial: every compute warp has written its own
        wait_on(&sh.red_bar[slot], par2);
        RowAcc r;
        r.init();
        if (lane < n_compute_warps) r = sh.warp_scratch[slot][lane];
        r = warp_reduce_two_step(r);
        // S[n, y] is sent by the CTA whose slice contains its vector (the last CTA for the scalar
        // tail); that CTA fetched it from global memory at the top of the step
        const int64_t yv = y / P;
        const bool mine = yv < nvec ? (yv >= v_lo && yv < v_lo + my_vecs) : owns_tail;
        // lane j sends this CTA's partial (and the token's logit) to CTA j
        // every CTA (this one included) receives 20 bytes from each CTA and 4 from the token's owner
        if (lane == 0) mbar_expect_tx(smem_u32(&sh.xchg_bar[slot]), csize * 20u + 4u);
        if (lane < (int)csize) {
          const uint32_t bar = map_to_cta(smem_u32(&sh.xchg_bar[slot]), (uint32_t)lane);
          st_async_v4(map_to_cta(smem_u32(&sh.partial4[slot][rank]), (uint32_t)lane), r.ms, r.zs, r.as, r.mt, bar);
          st_async_f32(map_to_cta(smem_u32(&sh.partial_zt[slot][rank]), (uint32_t)lane), r.zt, bar);
          if (mine) st_async_f32(map_to_cta(smem_u32(&sh.token_logit[slot]), (uint32_t)lane), sy, bar);
        }
      }
      // look ahead: row k + 2 goes into the buffer of row k - 1 once its gradient sweep is done
      row_n = row_l >= 0 ? next_row(cf_n) : -1;
      if (row_n >= 0) {
        if (row_g >= 0) wait_on(&sh.free_bar[buf_g], ((k - 1) / kSliceBufs) & 1u);
        if (lane == 0) issue_row(row_n, (k + 2) % kSliceBufs);
      }
      // finish the exchange of row k: row constants, identical in every CTA
      if (row_r >= 0) {
        if (ok) ok = mbar_wait_cluster_bounded(smem_u32(&sh.xchg_bar[slot]), par2);
        RowAcc r;
        r.init();
        if (lane < (int)csize) {
          const float4 p4 = sh.partial4[slot][lane];
          r.ms = p4.x;
          r.zs = p4.y;
          r.as = p4.z;
          r.mt = p4.w;
          r.zt = sh.partial_zt[slot][lane];
        }
        r = warp_reduce_two_step(r);
        const float gs = logf(r.zs), gt = logf(r.zt);
        const float ls = r.ms + gs, lt = r.mt + gt;
        const float kl = r.as / r.zs - ((r.ms - r.mt) + (gs - gt));
        const float d = ((sh.token_logit[slot] - r.ms) - gs) - b;
        if (lane == 0) {
          sh.grad_row[slot] = make_grad_row(make_float4(ls, lt, kl, d), cf_r, a.lambda, y);
          sh.row_after_next[slot] = row_n;
          const int64_t yl = y / P - v_lo;  // the token's vector within this CTA's slice, if it is here
          const bool here = yl >= 0 && yl < my_vecs;
          sh.token_patch[slot] = make_int2(here ? (int)(yl % n_compute) : -1,
                                           here ? (int)(((int64_t)y - v_lo * P) * E::kBytes) : 0);
          mbar_arrive(smem_u32(&sh.grad_bar[slot]));
          if (rank == 0) reinterpret_cast<float4 *>(a.row_ws)[row_r] = make_float4(ls, lt, kl, d);
        }
      }
    } else {
      // =================================================== compute warps
      if (row_r >= 0) {
        const uint32_t s_base = data_base + buf_r * 2u * slice_bytes, t_base = s_base + slice_bytes;
        if (my_vecs > 0) wait_on(&sh.load_bar[buf_r], (k / kSliceBufs) & 1u);
        RowAcc sweep;
        sweep.init();
        for (int i = ctid; i < my_vecs; i += n_compute) {
          float s[P], t[P];
          E::unpack(lds128(s_base + (uint32_t)i * 16u), s);
          E::unpack(lds128(t_base + (uint32_t)i * 16u), t);
          sweep.add<P>(s, t);
        }
        if (has_tail) {
          const char *srow = reinterpret_cast<const char *>(c.student) + row_r * row_bytes;
          const char *trow = reinterpret_cast<const char *>(c.teacher) + row_r * row_bytes;
          sweep.add1(E::load1(srow, tail_idx), E::load1(trow, tail_idx));
        }
        const RowAcc acc = warp_reduce_two_step(sweep);
        if (lane == 0) {
          sh.warp_scratch[slot][(tid >> 5) - 1] = acc;
          mbar_arrive(smem_u32(&sh.red_bar[slot]));
        }
      }
      if (row_g >= 0) {
        const uint32_t s_base = data_base + buf_g * 2u * slice_bytes, t_base = s_base + slice_bytes;
        wait_on(&sh.grad_bar[slot ^ 1u], ((k - 1) >> 1) & 1u);
        const GradRow gr = sh.grad_row[slot ^ 1u];
        char *orow = reinterpret_cast<char *>(a.dlogits) + row_g * row_bytes;
        uint4 *o4 = reinterpret_cast<uint4 *>(orow) + v_lo;
        for (int i = ctid; i < my_vecs; i += n_compute) {
          const uint4 sv = lds128(s_base + (uint32_t)i * 16u), tv = lds128(t_base + (uint32_t)i * 16u);
          st_stream(o4 + i, grad_vec<DT>(sv, tv, gr));
        }
        {
          // the stored token's element gets its extra term from the thread that wrote its vector
          // (same thread, so the two stores to that address stay in order)
          const int2 patch = sh.token_patch[slot ^ 1u];
          if (patch.x == ctid) {
            const float s = lds_logit<DT>(s_base + (uint32_t)patch.y), t = lds_logit<DT>(t_base + (uint32_t)patch.y);
            E::store1(orow, gr.y, fmaf(ex2(fmaf(s, kLog2e, gr.e0)), (s - t) - gr.K, gr.cg));
          }
        }
        if (has_tail) {
          const char *srow = reinterpret_cast<const char *>(c.student) + row_g * row_bytes;
          const char *trow = reinterpret_cast<const char *>(c.teacher) + row_g * row_bytes;
          const float s = E::load1(srow, tail_idx), t = E::load1(trow, tail_idx);
          float o = ex2(fmaf(s, kLog2e, gr.e0)) * ((s - t) - gr.K);
          if (tail_idx == gr.y) o += gr.cg;
          E::store1(orow, tail_idx, o);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive_relaxed(smem_u32(&sh.free_bar[buf_g]));
      }
      // The control warp scans ahead; the compute warps learn row k + 1 from the constants of
      // row k - 1 (read above) and give the rows passed over in between their zeros.
      if (k == 0) {
        row_n = row_l;  // found by every thread before the loop
      } else if (row_g >= 0) {
        row_n = sh.row_after_next[slot ^ 1u];
        if (row_r >= 0) {
          const int64_t stop = row_n >= 0 ? row_n : c.n_rows;
          for (int64_t n = row_r + n_clusters; n < stop; n += n_clusters) zero_row(n);
        }
      }
    }
    row_g = row_r;
    if (control) {
      row_r = row_l;
      cf_r = cf_l;
      row_l = row_n;
      cf_l = cf_n;
    } else {
      row_r = k == 0 ? row_l : row_n;  // compute warps run one row behind the control warp's scan
    }
  }

  if (!ok) sh.failed = 1;
  __syncthreads();
  if (tid == 0 && sh.failed && a.status) atomicOr(a.status, FOPD_DEV_TIMEOUT);
  // No CTA may exit while a peer can still write into its shared memory.
  cluster_arrive();
  cluster_wait();
}

}  // namespace fopd
