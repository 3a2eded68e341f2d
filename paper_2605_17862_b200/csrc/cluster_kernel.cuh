// Fused loss forward + backward with the row resident on chip (sm_100a).
//
// A thread-block cluster owns one token row at a time.  Each CTA of the
// cluster lands its slice of the student and teacher rows in shared memory
// with bulk asynchronous copies (global -> shared, completion on an mbarrier).
// The compute threads sweep the slice for the row's partial sums (maximum
// first, then the exponentials: no rescaling inside the sweep) and keep their
// student vectors in registers, so the student part of the buffer goes back at
// once; the teacher slice stays in its buffer until the gradient has been
// formed.  The CTAs exchange their partial sums through distributed shared
// memory; once all partials have landed every CTA holds the row's normalisers
// and KL, and the gradient is formed from the student registers and the teacher
// slice and streamed out.  Student and teacher logits are read from HBM once and
// dlogits written once: 3 * V * e bytes per differentiated row.
//
// Warp 0 of each CTA is a control warp, the other W (19 to 23) warps compute.  The rows of a
// cluster move through a software pipeline over two student and three teacher
// buffers per CTA; a compute thread holds the student vectors of two rows:
//
//   compute warps, step k:  sums of row k (student buffer k % 2 -> registers X,
//                           released; teacher buffer k % 3), posted to the control
//                           warp; gradient of row k - 1 from
//                           registers Y and teacher buffer (k - 1) % 3, which is then
//                           released; Y <- X
//   control warp,  step k:  start the student copy of row k + 2 into the buffer row k
//                           has left; merge the warps' partials of row k and send
//                           the CTA's to the cluster; when all CTAs' partials of row
//                           k are here, form the row constants for its gradient;
//                           start the teacher copy of row k + 2 into the buffer row
//                           k - 1 has left
//
// so the cluster exchange of row k is covered by the gradient of row k - 1 and the
// sums of row k + 1.  All hand-offs inside a CTA and between CTAs go through mbarriers (no
// CTA-wide or cluster-wide barrier inside the loop).  A small kernel run first
// writes each row's weight coef_i (0 for rows that are not differentiated), which
// lets the control warp look for rows with independent loads; the zeros of those
// rows are written by a kernel that runs beside this one.
//
// Every mbarrier wait is bounded.  A wait that runs out raises a flag in shared
// memory; every thread of the CTA looks at the flag once per step and leaves the row
// loop, the control warp waits (bounded again) for the copies it still has in
// flight, FOPD_DEV_TIMEOUT is recorded in the status word and the kernel ends (the
// results of that call are void).
#pragma once

#include "stream_kernels.cuh"

namespace fopd {

// Compute warps per CTA (W) and vectors of a row's slice a compute thread takes (NV; it holds
// the student vectors of two rows).  Every compute thread works through NV slots whether it has
// a vector for the last one or not, so the launcher picks the pair with the least padding.
#define FOPD_FUSED_SHAPES(X) X(1, 19) X(2, 19) X(3, 19) X(1, 21) X(2, 21) X(3, 21) X(1, 23) X(2, 23) X(3, 23)
constexpr int kFusedMaxNV = 3, kFusedMaxWarps = 23;
constexpr int kMaxClusterSize = 16;
constexpr int kStudentBufs = 2, kTeacherBufs = 3;
constexpr int kSliceBufs = kStudentBufs + kTeacherBufs;  // slices of shared memory per CTA
constexpr long long kWaitCycles = 200000000;  // SM cycles one mbarrier wait may take before giving up (~0.1 s)
// A logit below every real one, as a 32-bit pattern that reads the same way as one fp32 or as
// two bf16: register slots a thread has no vector for are filled with it, so that they add
// nothing to the sums (e^(x - max) = 0, x_s - x_t = 0) and need no branch.
constexpr uint32_t kNoLogitBits = 0xff7fff7fu;

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
// Arrival with release semantics (the default): what the arriving thread read or wrote before
// it is ordered before whatever the thread that sees the phase complete does next.  Slice
// buffers are handed back with it (the warp's reads of the buffer, then the arrival; the control
// warp starts the copy that overwrites the buffer only after it has seen the phase complete).
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
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
// Bounded waits: false if the phase did not complete within `limit` SM cycles.  try_wait itself
// parks the thread for a while, so the loop is kept to the poll and a branch; the clock is
// read once per kPollsPerClock polls.
constexpr int kPollsPerClock = 64;
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, long long limit) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  do {
    for (int i = 0; i < kPollsPerClock; ++i)
      if (mbar_try_wait(bar, parity)) return true;
  } while (clock64() - t0 <= limit);
  return false;
}
// The same for a warp whose polls should not take issue slots from its neighbours.
__device__ __forceinline__ bool mbar_wait_bounded_sleeping(uint32_t bar, uint32_t parity, long long limit) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  do {
    for (int i = 0; i < kPollsPerClock; ++i) {
      __nanosleep(64);
      if (mbar_try_wait(bar, parity)) return true;
    }
  } while (clock64() - t0 <= limit);
  return false;
}
__device__ __forceinline__ bool mbar_wait_cluster_bounded(uint32_t bar, uint32_t parity, long long limit) {
  if (mbar_try_wait_cluster(bar, parity)) return true;
  const long long t0 = clock64();
  do {
    for (int i = 0; i < kPollsPerClock; ++i) {
      __nanosleep(64);
      if (mbar_try_wait_cluster(bar, parity)) return true;
    }
  } while (clock64() - t0 <= limit);
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
// Barrier of all threads of the CTA that warps in different roles reach from different places.
template <int kThreads>
__device__ __forceinline__ void role_sync() {
  asm volatile("bar.sync 1, %0;" ::"n"(kThreads) : "memory");
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

// The same for lanes that already share their maxima: the sums add up as they are.
__device__ __forceinline__ RowAcc warp_sum_common_scale(RowAcc a) {
  const bool odd = threadIdx.x & 1;
  const float give = odd ? a.zs : a.as, keep = odd ? a.as : a.zs;  // even lanes collect zs, odd lanes as
  float za = keep + __shfl_xor_sync(0xffffffffu, give, 1);
  float zt = a.zt + __shfl_xor_sync(0xffffffffu, a.zt, 1);
#pragma unroll
  for (int off = 2; off < 32; off <<= 1) {
    za += __shfl_xor_sync(0xffffffffu, za, off);
    zt += __shfl_xor_sync(0xffffffffu, zt, off);
  }
  const float other = __shfl_xor_sync(0xffffffffu, za, 1);
  a.zs = odd ? other : za;
  a.as = odd ? za : other;
  a.zt = zt;
  return a;
}

// Largest logit of N 16-byte vectors.  bf16: packed maxima over all words first, then the two
// halves of the one word that is left.
template <int DT, int N>
__device__ __forceinline__ float vecs_max(const uint4 (&v)[N]) {
  if (DT == FOPD_BF16) {
    __nv_bfloat162 m;
#pragma unroll
    for (int j = 0; j < N; ++j) {
      const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162 *>(&v[j].x),
                           b = *reinterpret_cast<const __nv_bfloat162 *>(&v[j].y),
                           c = *reinterpret_cast<const __nv_bfloat162 *>(&v[j].z),
                           d = *reinterpret_cast<const __nv_bfloat162 *>(&v[j].w);
      const __nv_bfloat162 mj = __hmax2(__hmax2(a, b), __hmax2(c, d));
      m = j == 0 ? mj : __hmax2(m, mj);
    }
    const uint32_t w = *reinterpret_cast<const uint32_t *>(&m);
    return fmaxf(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
  }
  float m = -INFINITY;
#pragma unroll
  for (int j = 0; j < N; ++j)
    m = fmaxf(fmaxf(max3(__uint_as_float(v[j].x), __uint_as_float(v[j].y), __uint_as_float(v[j].z)), __uint_as_float(v[j].w)), m);
  return m;
}

// Packed single precision: two fp32 values in one 64-bit register, one instruction for both
// (sm_100a add / sub / mul / fma on .f32x2).  The sweeps over registers are bound by the
// special-function pipe and instruction issue together; halving the arithmetic instructions
// around the exponentials is what lets the two overlap.
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float a, float b) {
  f32x2 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void unpack2(f32x2 r, float &a, float &b) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(r));
}
__device__ __forceinline__ f32x2 sub2(f32x2 a, f32x2 b) {
  f32x2 r;
  asm("sub.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) {
  f32x2 r;
  asm("add.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) {
  f32x2 r;
  asm("mul.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
  f32x2 r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
__device__ __forceinline__ f32x2 ex2_2(f32x2 x) {
  float a, b;
  unpack2(x, a, b);
  return pack2(ex2(a), ex2(b));
}
// The logits of a 16-byte vector as packed pairs (element 2q in the low half of pair q).
template <int DT>
struct Pairs;
template <>
struct Pairs<FOPD_BF16> {
  static constexpr int kPairs = 4;
  __device__ static __forceinline__ void get(const uint4 &v, f32x2 (&p)[4]) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) p[q] = pack2(__uint_as_float(w[q] << 16), __uint_as_float(w[q] & 0xffff0000u));
  }
  __device__ static __forceinline__ uint4 put(const f32x2 (&p)[4]) {
    uint32_t w[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      float a, b;
      unpack2(p[q], a, b);
      __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
      w[q] = *reinterpret_cast<uint32_t *>(&h);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
  }
};
template <>
struct Pairs<FOPD_F32> {
  static constexpr int kPairs = 2;
  __device__ static __forceinline__ void get(const uint4 &v, f32x2 (&p)[2]) {
    p[0] = pack2(__uint_as_float(v.x), __uint_as_float(v.y));
    p[1] = pack2(__uint_as_float(v.z), __uint_as_float(v.w));
  }
  __device__ static __forceinline__ uint4 put(const f32x2 (&p)[2]) {
    float a, b, c, d;
    unpack2(p[0], a, b);
    unpack2(p[1], c, d);
    return make_uint4(__float_as_uint(a), __float_as_uint(b), __float_as_uint(c), __float_as_uint(d));
  }
};

// Weight of every row of a chunk, written before the on-chip kernel: coef of its sample if the
// row is differentiated (aligned, ids in range, coef > 0), else 0.  Reports bad ids in the
// status word.
static __global__ void __launch_bounds__(256)
    row_weight_kernel(ChunkDev c, int32_t B, const float *coef, int32_t *status, float *row_cf) {
  const int64_t n = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (n >= c.n_rows) return;
  float cf = 0.f;
  if (row_is_aligned(c, n, B, status, true)) cf = coef[c.sid[n]];
  row_cf[n] = cf > 0.f ? cf : 0.f;
}

// Zeros for the rows the on-chip kernel does not differentiate, so that the on-chip kernel only
// ever sees rows it works on.  A CTA is one warp with a 48 KB buffer of zeros in shared memory;
// one lane writes a row with bulk asynchronous copies shared -> global, which take no further
// instructions.  Launched AFTER the on-chip kernel with programmatic stream serialisation: the
// on-chip kernel lets its dependents go at once, so these CTAs run on the SMs its clusters leave
// free (13 of 148 with clusters of nine) while it works and on all SMs once it has ended.  The
// buffer is larger than what an SM's shared-memory configuration leaves beside an on-chip CTA
// (the configurations are at most 36 KB apart), on purpose: zero-fill CTAs that shared an SM with
// on-chip CTAs slowed those down by more than they gained (measured with 16 KB buffers; 32, 40
// and 48 KB are within 1 % of each other, 48 first).  The
// two kernels write disjoint rows.  CTA 0 ends by waiting for the on-chip kernel, so that this
// grid -- which is what the next launch in the stream waits for -- is not complete before the
// on-chip kernel is.
constexpr uint32_t kZeroBufBytes = 49152;
template <int DT>
__global__ void __launch_bounds__(32) zero_rows_kernel(ChunkDev c, const float *row_cf, void *dlogits) {
  using E = Elem<DT>;
  extern __shared__ __align__(128) unsigned char zero_buf[];
  const int lane = threadIdx.x;
  const int64_t pitch = c.stride * E::kBytes;
  const int64_t bulk_bytes = (c.vocab * E::kBytes) & ~int64_t(15);  // the rest of a row (< 16 bytes) by plain stores
  bool ready = false;
  for (int64_t n = blockIdx.x; n < c.n_rows; n += gridDim.x) {
    if (row_cf[n] > 0.f) continue;
    if (!ready) {
      for (uint32_t i = lane * 16u; i < kZeroBufBytes; i += 32u * 16u)
        *reinterpret_cast<uint4 *>(zero_buf + i) = make_uint4(0u, 0u, 0u, 0u);
      // the zeros were written through the generic proxy; the copies read them through the async proxy
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      ready = true;
    }
    char *orow = reinterpret_cast<char *>(dlogits) + n * pitch;
    if (lane == 0) {
      const uint32_t src = smem_u32(zero_buf);
      for (int64_t off = 0; off < bulk_bytes; off += kZeroBufBytes) {
        const uint32_t bytes = (uint32_t)min((int64_t)kZeroBufBytes, bulk_bytes - off);
        asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(orow + off), "r"(src), "r"(bytes)
                     : "memory");
      }
      asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    }
    const int64_t tail = bulk_bytes / E::kBytes + lane;
    if (tail < c.vocab) E::store1(orow, tail, 0.f);
  }
  // the buffer must outlive the copies that read it; they are this thread's own and always complete
  if (ready && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  if (blockIdx.x == 0) asm volatile("griddepcontrol.wait;" ::: "memory");
}

// What the control warp hands the compute warps for the gradient of one row.
struct __align__(16) RowRec {
  float e0, K, cg;        // see GradRow
  int32_t y;              // the stored token's column
  int32_t y_owner;        // compute thread that holds the token's vector, or -1 (not in this CTA's slice)
  int32_t y_j, y_e;       // which of that thread's vectors, which element of the vector
  int32_t pad;
  long long after_next;   // the cluster's differentiated row after the next one, or -1
  long long pad2;
};

struct ClusterShared {
  unsigned long long load_s_bar[kStudentBufs];  // student slice landed (1 arrival + bytes)
  unsigned long long load_t_bar[kTeacherBufs];  // teacher slice landed (1 arrival + bytes)
  unsigned long long free_s_bar[kStudentBufs];  // student slice copied into registers (one arrival per compute warp)
  unsigned long long free_t_bar[kTeacherBufs];  // teacher slice no longer needed (one arrival per compute warp)
  unsigned long long red_bar[2];             // [row parity] warp partials written (one arrival per compute warp)
  unsigned long long grad_bar[2];            // [row parity] rec ready (1 arrival)
  uint4 no_logit;                            // filler for register slots without a vector
  unsigned long long xchg_bar[2];            // [row parity] partials of all CTAs here (1 arrival + bytes)
  float4 partial4[2][kMaxClusterSize];       // [row parity][source CTA rank] {ms, zs, as, mt}, written by peers
  float partial_zt[2][kMaxClusterSize];      // [row parity][source CTA rank] zt
  float token_logit[2];                      // [row parity] S[n, y_n], written by the CTA whose slice holds it
  RowAcc warp_scratch[2][kFusedMaxWarps];    // [row parity][compute warp]
  RowRec rec[2];                             // [row parity]
  long long first_rows[2];                   // the cluster's first two differentiated rows (or -1)
  int failed;                                // a bounded wait ran out somewhere in this CTA
};

struct FusedArgs {
  ChunkDev c;
  float lambda;
  void *dlogits;
  const float *row_cf;  // [n_rows] from row_weight_kernel
  float *row_ws;        // [n_rows,4] out: {lse_s, lse_t, kl, d} of the differentiated rows
  int32_t *status;
  int slice_vecs;       // 16-byte vectors of a row per CTA (the last CTAs' slices may be shorter or empty)
  long long wait_cycles;  // limit of one mbarrier wait
};

template <int DT, int NV, int W>
__global__ void __launch_bounds__(W * 32 + 32, 1) fused_cluster_kernel(FusedArgs a) {
  constexpr int kFusedComputeWarps = W, kFusedCompute = W * 32, kFusedThreads = W * 32 + 32;
  using E = Elem<DT>;
  using PP = Pairs<DT>;
  constexpr int P = E::kPerVec;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  ClusterShared &sh = *reinterpret_cast<ClusterShared *>(smem_raw);
  const uint32_t data_off = (sizeof(ClusterShared) + 127u) & ~127u;
  const uint32_t slice_bytes = (uint32_t)a.slice_vecs * 16u;
  // student buffers first, then the teacher buffers
  const uint32_t s_bufs = smem_u32(smem_raw) + data_off, t_bufs = s_bufs + kStudentBufs * slice_bytes;

  const uint32_t rank = cluster_ctarank(), csize = cluster_nctarank();
  const int64_t n_clusters = gridDim.x / csize, cluster_id = blockIdx.x / csize;
  const ChunkDev &c = a.c;
  const int64_t V = c.vocab, nvec = V / P;
  const int tid = threadIdx.x, lane = tid & 31;
  const bool control = tid < 32;
  const int ctid = tid - 32;   // index among the compute threads (negative in the control warp)
  const long long limit = a.wait_cycles;

  // This CTA's slice of every row, in vectors; compute thread t takes vectors t, t + kFusedCompute, ...
  const int64_t v_lo = (int64_t)rank * a.slice_vecs;
  const int my_vecs = (int)max((int64_t)0, min((int64_t)a.slice_vecs, nvec - v_lo));
  const int nv = control ? 0 : max(0, min(NV, (my_vecs - ctid + kFusedCompute - 1) / kFusedCompute));
  const bool owns_tail = (rank == csize - 1);
  const int64_t tail_idx = nvec * P + ctid;  // scalar tail element handled by the last CTA's compute threads
  const bool has_tail = owns_tail && !control && tail_idx < V;
  const int64_t row_bytes = c.stride * E::kBytes;

  // the kernel that writes the zeros of the other rows may start now (it needs nothing from here)
  asm volatile("griddepcontrol.launch_dependents;");
  if (tid == 0) {
    for (int b = 0; b < kStudentBufs; ++b) {
      mbar_init(smem_u32(&sh.load_s_bar[b]), 1);
      mbar_init(smem_u32(&sh.free_s_bar[b]), kFusedComputeWarps);
    }
    for (int b = 0; b < kTeacherBufs; ++b) {
      mbar_init(smem_u32(&sh.load_t_bar[b]), 1);
      mbar_init(smem_u32(&sh.free_t_bar[b]), kFusedComputeWarps);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&sh.red_bar[b]), kFusedComputeWarps);
      mbar_init(smem_u32(&sh.grad_bar[b]), 1);
      mbar_init(smem_u32(&sh.xchg_bar[b]), 1);
      RowRec r0 = {};
      r0.y_owner = -1;
      r0.after_next = -1;
      sh.rec[b] = r0;
      sh.first_rows[b] = -1;
    }
    sh.no_logit = make_uint4(kNoLogitBits, kNoLogitBits, kNoLogitBits, kNoLogitBits);
    sh.failed = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  cluster_arrive();
  cluster_wait();

  volatile int *failed = &sh.failed;

  if (control) {
    // =================================================================== control warp
    auto wait_on = [&](unsigned long long *bar, uint32_t parity) -> bool {
      if (mbar_wait_bounded(smem_u32(bar), parity, limit)) return true;
      *failed = 1;
      return false;
    };
    // One lane starts the copy of the student / teacher slice of row number kk (row n).
    auto issue_s = [&](int64_t n, uint32_t kk) {
      if (my_vecs == 0) return;
      const uint32_t b = kk % kStudentBufs, bytes = (uint32_t)my_vecs * 16u, bar = smem_u32(&sh.load_s_bar[b]);
      mbar_expect_tx(bar, bytes);
      bulk_load(s_bufs + b * slice_bytes, reinterpret_cast<const char *>(c.student) + n * row_bytes + v_lo * 16, bytes, bar);
    };
    auto issue_t = [&](int64_t n, uint32_t kk) {
      if (my_vecs == 0) return;
      const uint32_t b = kk % kTeacherBufs, bytes = (uint32_t)my_vecs * 16u, bar = smem_u32(&sh.load_t_bar[b]);
      mbar_expect_tx(bar, bytes);
      bulk_load(t_bufs + b * slice_bytes, reinterpret_cast<const char *>(c.teacher) + n * row_bytes + v_lo * 16, bytes, bar);
    };
    // Next differentiated row of this cluster (-1 when the rows are exhausted).  The 32 lanes
    // hold the weights of a window of 32 of the cluster's rows; a window is loaded once and its
    // hits are handed out one by one.
    int64_t win_n = cluster_id;   // first row of the window
    float win_cf = 0.f;
    unsigned win_hits = 0;        // lanes of the window whose rows are still to be handed out
    bool win_loaded = false;
    auto next_row = [&](float &cf_out) -> int64_t {
      for (;;) {
        if (!win_loaded) {
          if (win_n >= c.n_rows) {
            cf_out = 0.f;
            return -1;
          }
          const int64_t n = win_n + (int64_t)lane * n_clusters;
          win_cf = n < c.n_rows ? __ldg(a.row_cf + n) : 0.f;
          win_hits = __ballot_sync(0xffffffffu, win_cf > 0.f);
          win_loaded = true;
        }
        if (win_hits) {
          const int l = __ffs(win_hits) - 1;
          win_hits &= win_hits - 1;
          cf_out = __shfl_sync(0xffffffffu, win_cf, l);
          return win_n + (int64_t)l * n_clusters;
        }
        win_n += 32 * n_clusters;
        win_loaded = false;
      }
    };

    // rows k .. k + 3 of the pipeline and their weights; the first copies go out at once
    float cf0 = 0.f, cf1 = 0.f, cf2 = 0.f, cf3 = 0.f;
    int64_t q0 = next_row(cf0);
    int64_t q1 = q0 >= 0 ? next_row(cf1) : -1;
    int64_t q2 = q1 >= 0 ? next_row(cf2) : -1;
    int64_t q3 = q2 >= 0 ? next_row(cf3) : -1;
    uint32_t issued_s = 0, issued_t = 0;  // lane 0: rows whose student / teacher copy has been started
    if (lane == 0) {
      if (q0 >= 0) issue_s(q0, 0), issue_t(q0, 0), issued_s = 1, issued_t = 1;
      if (q1 >= 0) issue_s(q1, 1), issue_t(q1, 1), issued_s = 2, issued_t = 2;
      if (q2 >= 0) issue_t(q2, 2), issued_t = 3;
      sh.first_rows[0] = q0;
      sh.first_rows[1] = q1;
    }
    role_sync<kFusedThreads>();  // the compute warps learn the first rows

    bool ok = true;
    for (uint32_t k = 0; q0 >= 0; ++k) {
      if (*failed) {
        ok = false;
        break;
      }
      const uint32_t slot = k & 1u, par2 = (k >> 1) & 1u;
      // side inputs of row k, used after the waits below (row weights > 0 imply a token in range)
      const int32_t y = c.tokens[q0];
      const float b = c.behav[q0];
      const float sy = E::load1(reinterpret_cast<const char *>(c.student) + q0 * row_bytes, y);
      // row k + 4, looked up now so that the load it takes is off the path of the waits
      float cf4 = 0.f;
      const int64_t q4 = q3 >= 0 ? next_row(cf4) : -1;
      // the compute warps copy the student slice of row k into registers first thing: row k + 2
      // takes its buffer
      if (q2 >= 0) {
        if (!(ok = wait_on(&sh.free_s_bar[k % kStudentBufs], (k / kStudentBufs) & 1u))) break;
        if (lane == 0) issue_s(q2, k + 2), issued_s = k + 3;
      }
      // CTA partial: every compute warp has written its own
      if (!(ok = wait_on(&sh.red_bar[slot], par2))) break;
      RowAcc r;
      r.init();
      if (lane < kFusedComputeWarps) r = sh.warp_scratch[slot][lane];
      r = warp_reduce_two_step(r);
      // S[n, y] is sent by the CTA whose slice contains its vector (the last CTA for the scalar
      // tail); that CTA fetched it from global memory above
      const int64_t yv = y / P;
      const bool mine = yv < nvec ? (yv >= v_lo && yv < v_lo + my_vecs) : owns_tail;
      // lane j sends this CTA's partial (and the token's logit) to CTA j: every CTA (this one
      // included) receives 20 bytes from each CTA and 4 from the token's owner
      if (lane == 0) mbar_expect_tx(smem_u32(&sh.xchg_bar[slot]), csize * 20u + 4u);
      if (lane < (int)csize) {
        const uint32_t bar = map_to_cta(smem_u32(&sh.xchg_bar[slot]), (uint32_t)lane);
        st_async_v4(map_to_cta(smem_u32(&sh.partial4[slot][rank]), (uint32_t)lane), r.ms, r.zs, r.as, r.mt, bar);
        st_async_f32(map_to_cta(smem_u32(&sh.partial_zt[slot][rank]), (uint32_t)lane), r.zt, bar);
        if (mine) st_async_f32(map_to_cta(smem_u32(&sh.token_logit[slot]), (uint32_t)lane), sy, bar);
      }
      // the exchange of row k: row constants, identical in every CTA
      if (!mbar_wait_cluster_bounded(smem_u32(&sh.xchg_bar[slot]), par2, limit)) {
        *failed = 1;
        ok = false;
        break;
      }
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
        const GradRow g = make_grad_row(make_float4(ls, lt, kl, d), cf0, a.lambda, y);
        const int64_t yl = yv - v_lo;  // the token's vector within this CTA's slice, if it is here
        const bool here = yv < nvec && yl >= 0 && yl < my_vecs;
        RowRec &rec = sh.rec[slot];
        *reinterpret_cast<float4 *>(&rec.e0) = make_float4(g.e0, g.K, g.cg, __int_as_float(y));
        *reinterpret_cast<int4 *>(&rec.y_owner) =
            make_int4(here ? (int)(yl % kFusedCompute) : -1, here ? (int)(yl / kFusedCompute) : 0, (int)(y % P), 0);
        rec.after_next = q2;
        mbar_arrive(smem_u32(&sh.grad_bar[slot]));
        if (rank == 0) reinterpret_cast<float4 *>(a.row_ws)[q0] = make_float4(ls, lt, kl, d);
      }
      // during this step the gradient of row k - 1 is formed; when it is done the teacher copy of
      // row k + 2 takes the buffer row k - 1 has left
      if (k >= 1 && q2 >= 0) {
        if (!(ok = wait_on(&sh.free_t_bar[(k + 2) % kTeacherBufs], ((k - 1) / kTeacherBufs) & 1u))) break;
        if (lane == 0) issue_t(q2, k + 2), issued_t = k + 3;
      }
      q0 = q1;
      cf0 = cf1;
      q1 = q2;
      cf1 = cf2;
      q2 = q3;
      cf2 = cf3;
      q3 = q4;
      cf3 = cf4;
    }
    // Nothing may be left in flight into this CTA's shared memory when it exits: on the normal
    // path every copy has been waited for by the compute warps; after a failed wait the copies
    // started last are waited for here (bounded).
    if (!ok && my_vecs > 0) {
      const uint32_t ns = __shfl_sync(0xffffffffu, issued_s, 0), nt = __shfl_sync(0xffffffffu, issued_t, 0);
      for (uint32_t j = ns > kStudentBufs ? ns - kStudentBufs : 0; j < ns; ++j)
        (void)mbar_wait_bounded(smem_u32(&sh.load_s_bar[j % kStudentBufs]), (j / kStudentBufs) & 1u, limit);
      for (uint32_t j = nt > kTeacherBufs ? nt - kTeacherBufs : 0; j < nt; ++j)
        (void)mbar_wait_bounded(smem_u32(&sh.load_t_bar[j % kTeacherBufs]), (j / kTeacherBufs) & 1u, limit);
    }
  } else {
    // =================================================================== compute warps
    auto wait_on = [&](unsigned long long *bar, uint32_t parity) -> bool {
      if (mbar_wait_bounded(smem_u32(bar), parity, limit)) return true;
      *failed = 1;
      return false;
    };
    role_sync<kFusedThreads>();  // the control warp has found the first rows
    const uint32_t no_logit = smem_u32(&sh.no_logit);
    // Shared-memory address of this thread's j-th vector inside a slice buffer (the filler for
    // slots without a vector).
    uint32_t voff[NV];
#pragma unroll
    for (int j = 0; j < NV; ++j) voff[j] = (uint32_t)(ctid + j * kFusedCompute) * 16u;

    int64_t cur = sh.first_rows[0], prev = -1;
    const int64_t second = sh.first_rows[1];

    uint4 X[NV], Y[NV];          // student vectors of row k and of row k - 1
    float x_tail_s = 0.f, x_tail_t = 0.f, y_tail_s = 0.f, y_tail_t = 0.f;
    for (uint32_t k = 0; cur >= 0 || prev >= 0; ++k) {
      if (*failed) break;
      const uint32_t slot = k & 1u;
      if (cur >= 0) {
        // ---- sums of row k.  Student vectors into registers, where they stay for the gradient;
        // teacher vectors are read again then.
        const uint32_t sb = k % kStudentBufs, tb = k % kTeacherBufs;
        if (my_vecs > 0 && (!wait_on(&sh.load_s_bar[sb], (k / kStudentBufs) & 1u) ||
                            !wait_on(&sh.load_t_bar[tb], (k / kTeacherBufs) & 1u)))
          break;
        const uint32_t s_base = s_bufs + sb * slice_bytes, t_base = t_bufs + tb * slice_bytes;
        uint4 T[NV];
        RowAcc acc;
        acc.init();
#pragma unroll
        for (int j = 0; j < NV; ++j) {
          X[j] = lds128(j < nv ? s_base + voff[j] : no_logit);
          T[j] = lds128(j < nv ? t_base + voff[j] : no_logit);
        }
        acc.ms = vecs_max<DT, NV>(X);
        acc.mt = vecs_max<DT, NV>(T);
        if (has_tail) {
          x_tail_s = E::load1(reinterpret_cast<const char *>(c.student) + cur * row_bytes, tail_idx);
          x_tail_t = E::load1(reinterpret_cast<const char *>(c.teacher) + cur * row_bytes, tail_idx);
          acc.ms = fmaxf(acc.ms, x_tail_s);
          acc.mt = fmaxf(acc.mt, x_tail_t);
        }
        // The warp agrees on its maxima before the exponentials, so that its lanes' sums are on one
        // scale and merge by plain additions: the chain of dependent steps after the sweep, which
        // all warps would sit through at the same time, shrinks to the shuffles.
        acc.ms = warp_max(acc.ms);
        acc.mt = warp_max(acc.mt);
        // the student slice is in registers now (the maxima have looked at all of it): its buffer
        // goes back (the warp-wide maximum has also brought the lanes together)
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&sh.free_s_bar[sb]));
        {
          // Exponent (x - max) * log2(e) in one fused multiply-add, x * log2(e) - c with c =
          // fl(max * log2(e)).  The product is exact inside the fma, so the result is off by the
          // rounding of c alone, c_lo = max * log2(e) - c, which the next fma gives exactly and
          // which is the same for every element of the warp: the sums come out scaled by
          // 2^c_lo and are put right afterwards (|c_lo| < 1e-4, so 2^-c_lo = 1 - c_lo ln 2 to
          // 1e-9).  The accuracy does not depend on the size of the logits.
          // (a warp with nothing but filler slots: its maximum is kept away from overflow in c)
          const float ms_f = fmaxf(acc.ms, -2e38f), mt_f = fmaxf(acc.mt, -2e38f);
          const float cs = ms_f * kLog2e, ct = mt_f * kLog2e;
          const float cs_lo = fmaf(ms_f, kLog2e, -cs), ct_lo = fmaf(mt_f, kLog2e, -ct);
          const f32x2 cs2 = pack2(-cs, -cs), ct2 = pack2(-ct, -ct), l2 = pack2(kLog2e, kLog2e);
          f32x2 zs2 = pack2(0.f, 0.f), as2 = zs2, zt2 = zs2;  // student and teacher sums take the same steps
#pragma unroll
          for (int j = 0; j < NV; ++j) {
            f32x2 s2[PP::kPairs], t2[PP::kPairs];
            PP::get(X[j], s2);
            PP::get(T[j], t2);
#pragma unroll
            for (int q = 0; q < PP::kPairs; ++q) {
              const f32x2 es = ex2_2(fma2(s2[q], l2, cs2)), et = ex2_2(fma2(t2[q], l2, ct2));
              zs2 = add2(zs2, es);
              as2 = fma2(es, sub2(s2[q], t2[q]), as2);
              zt2 = add2(zt2, et);
            }
          }
          const float fix_s = -cs_lo * kLn2, fix_t = -ct_lo * kLn2;
          float lo, hi;
          unpack2(zs2, lo, hi);
          acc.zs = fmaf(lo + hi, fix_s, lo + hi);
          unpack2(as2, lo, hi);
          acc.as = fmaf(lo + hi, fix_s, lo + hi);
          unpack2(zt2, lo, hi);
          acc.zt = fmaf(lo + hi, fix_t, lo + hi);
        }
        if (has_tail) {
          const float e = ex2((x_tail_s - acc.ms) * kLog2e);
          acc.zs += e;
          acc.as = fmaf(e, x_tail_s - x_tail_t, acc.as);
          acc.zt += ex2((x_tail_t - acc.mt) * kLog2e);
        }
        acc = warp_sum_common_scale(acc);
        if (lane == 0) {
          sh.warp_scratch[slot][ctid >> 5] = acc;
          mbar_arrive(smem_u32(&sh.red_bar[slot]));
        }
      }
      // row k + 1: from the prologue for the first step, from the constants of row k - 1 afterwards
      int64_t next = second;
      if (prev >= 0) {
        // ---- gradient of row k - 1 from the student registers and the teacher slice
        if (!wait_on(&sh.grad_bar[slot ^ 1u], ((k - 1) >> 1) & 1u)) break;
        GradRow gr;
        int y_owner, y_j, y_e;
        {
          const RowRec &rec = sh.rec[slot ^ 1u];
          const float4 c4 = *reinterpret_cast<const float4 *>(&rec.e0);   // e0, K, cg, y
          const int4 t4 = *reinterpret_cast<const int4 *>(&rec.y_owner);   // y_owner, y_j, y_e, pad
          gr.e0 = c4.x;
          gr.K = c4.y;
          gr.cg = c4.z;
          gr.y = __float_as_int(c4.w);
          y_owner = t4.x;
          y_j = t4.y;
          y_e = t4.z;
          next = rec.after_next;
        }
        const uint32_t tb = (k - 1) % kTeacherBufs, t_base = t_bufs + tb * slice_bytes;
        char *orow = reinterpret_cast<char *>(a.dlogits) + prev * row_bytes;
        uint4 *o4 = reinterpret_cast<uint4 *>(orow) + v_lo + ctid;
        const bool token_here = y_owner == ctid;
        const f32x2 l2g = pack2(kLog2e, kLog2e), e2g = pack2(gr.e0, gr.e0), K2g = pack2(gr.K, gr.K);
#pragma unroll
        for (int j = 0; j < NV; ++j) {
          f32x2 s2[PP::kPairs], t2[PP::kPairs], o2[PP::kPairs];
          PP::get(Y[j], s2);
          PP::get(lds128(j < nv ? t_base + voff[j] : no_logit), t2);
#pragma unroll
          for (int q = 0; q < PP::kPairs; ++q)
            o2[q] = mul2(ex2_2(fma2(s2[q], l2g, e2g)), sub2(sub2(s2[q], t2[q]), K2g));
          if (token_here && y_j == j) {
            // the stored token's element carries the anchor's extra term
#pragma unroll
            for (int q = 0; q < PP::kPairs; ++q) {
              float sa, sb, ta, tb2, oa, ob;
              unpack2(s2[q], sa, sb);
              unpack2(t2[q], ta, tb2);
              unpack2(o2[q], oa, ob);
              const bool odd = y_e & 1, hit = q == (y_e >> 1);
              const float sy = odd ? sb : sa, ty = odd ? tb2 : ta;
              const float oy = fmaf(ex2(fmaf(sy, kLog2e, gr.e0)), (sy - ty) - gr.K, gr.cg);
              o2[q] = pack2(hit && !odd ? oy : oa, hit && odd ? oy : ob);
            }
          }
          const uint4 o = PP::put(o2);
          if (j < nv) st_stream(o4 + j * kFusedCompute, o);
        }
        // the teacher slice has been read for the last time: its buffer goes back
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&sh.free_t_bar[tb]));
        if (has_tail) {
          float o = ex2(fmaf(y_tail_s, kLog2e, gr.e0)) * ((y_tail_s - y_tail_t) - gr.K);
          if (tail_idx == gr.y) o = fmaf(ex2(fmaf(y_tail_s, kLog2e, gr.e0)), (y_tail_s - y_tail_t) - gr.K, gr.cg);
          E::store1(orow, tail_idx, o);
        }
      }
      if (cur < 0) next = -1;
#pragma unroll
      for (int j = 0; j < NV; ++j) Y[j] = X[j];
      y_tail_s = x_tail_s;
      y_tail_t = x_tail_t;
      prev = cur;
      cur = next;
    }
  }

  __syncthreads();
  if (sh.failed) {
    if (tid == 0 && a.status) atomicOr(a.status, FOPD_DEV_TIMEOUT);
    // give stores that peers may still have in flight into this CTA's shared memory time to land
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000) {
    }
  }
  // No CTA may exit while a peer can still write into its shared memory.
  cluster_arrive();
  cluster_wait();
}

// Self-test of the bounded wait: one CTA initialises an mbarrier that expects two arrivals,
// arrives once and waits for at most `limit` SM cycles.  The phase cannot complete, so the wait
// must give up: the kernel records FOPD_DEV_TIMEOUT in the status word and returns.  Nothing
// here waits without a limit.
static __global__ void __launch_bounds__(32) bounded_wait_selftest_kernel(long long limit, int32_t *status,
                                                                          long long *waited_cycles) {
  __shared__ unsigned long long bar;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 2);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  if (threadIdx.x == 0) {
    mbar_arrive(smem_u32(&bar));
    const long long t0 = clock64();
    const bool done = mbar_wait_bounded(smem_u32(&bar), 0u, limit);
    if (waited_cycles) *waited_cycles = clock64() - t0;
    if (!done && status) atomicOr(status, FOPD_DEV_TIMEOUT);
  }
}

}  // namespace fopd
