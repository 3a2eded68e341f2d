// Shared device helpers of libfopd: packed-logit loads, online softmax
// accumulators and fixed-order block reductions.  sm_100a only.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/fopd.h"

namespace fopd {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kNegBig = -3.0e38f;  // "no element seen yet" marker for running maxima

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// max of three (one instruction on sm_100a)
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
template <int N>
__device__ __forceinline__ float max_of(const float (&x)[N]) {
  if (N == 8) return fmaxf(max3(x[0], x[1], x[2]), max3(x[3], x[4], max3(x[5], x[6], x[7 % N])));
  if (N == 4) return fmaxf(x[0], max3(x[1], x[2 % N], x[3 % N]));
  float v = x[0];
#pragma unroll
  for (int i = 1; i < N; ++i) v = fmaxf(v, x[i]);
  return v;
}

// Streaming (read-once) 16-byte global load.
__device__ __forceinline__ uint4 ld_stream(const void *p) {
  uint4 v;
  asm volatile("ld.global.cs.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

__device__ __forceinline__ void st_stream(void *p, uint4 v) {
  asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z),
               "r"(v.w)
               : "memory");
}

// Element traits: how many logits one 16-byte vector holds and how to unpack it.
template <int DT>
struct Elem;

template <>
struct Elem<FOPD_BF16> {
  static constexpr int kBytes = 2;
  static constexpr int kPerVec = 8;
  __device__ static __forceinline__ void unpack(const uint4 &v, float (&x)[8]) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      x[2 * i] = __uint_as_float(w[i] << 16);
      x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
  __device__ static __forceinline__ uint4 pack(const float (&x)[8]) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      __nv_bfloat162 h = __floats2bfloat162_rn(x[2 * i], x[2 * i + 1]);
      w[i] = *reinterpret_cast<uint32_t *>(&h);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
  }
  __device__ static __forceinline__ float load1(const void *base, int64_t idx) {
    return __uint_as_float(((uint32_t) reinterpret_cast<const uint16_t *>(base)[idx]) << 16);
  }
  __device__ static __forceinline__ void store1(void *base, int64_t idx, float x) {
    reinterpret_cast<__nv_bfloat16 *>(base)[idx] = __float2bfloat16_rn(x);
  }
};

template <>
struct Elem<FOPD_F32> {
  static constexpr int kBytes = 4;
  static constexpr int kPerVec = 4;
  __device__ static __forceinline__ void unpack(const uint4 &v, float (&x)[4]) {
    x[0] = __uint_as_float(v.x);
    x[1] = __uint_as_float(v.y);
    x[2] = __uint_as_float(v.z);
    x[3] = __uint_as_float(v.w);
  }
  __device__ static __forceinline__ uint4 pack(const float (&x)[4]) {
    return make_uint4(__float_as_uint(x[0]), __float_as_uint(x[1]), __float_as_uint(x[2]),
                      __float_as_uint(x[3]));
  }
  __device__ static __forceinline__ float load1(const void *base, int64_t idx) {
    return reinterpret_cast<const float *>(base)[idx];
  }
  __device__ static __forceinline__ void store1(void *base, int64_t idx, float x) {
    reinterpret_cast<float *>(base)[idx] = x;
  }
};

// Online accumulators of one row.  Student side: running max m, Z = sum e^{s-m},
// A = sum e^{s-m} (s - t).  Teacher side: running max and Z only.  From them
//   lse = m + log Z,   sum_v p_s(v) (s_v - t_v) = A / Z,
//   kl  = A / Z - lse_s + lse_t                       (Eq. 12, reverse KL).
struct RowAcc {
  float ms, zs, as, mt, zt;
  __device__ __forceinline__ void init() {
    ms = mt = kNegBig;
    zs = as = zt = 0.f;
  }
  // Merge another partial (order of the two operands does not change the
  // maxima; the sums are combined lower-index first by the callers).
  __device__ __forceinline__ void merge(const RowAcc &o) {
    const float Ms = fmaxf(ms, o.ms), Mt = fmaxf(mt, o.mt);
    const float ra = ex2((ms - Ms) * kLog2e), rb = ex2((o.ms - Ms) * kLog2e);
    // Explicit fma/mul so that student and teacher sums round identically
    // (teacher == student must give a KL of exactly zero).
    zs = __fmaf_rn(zs, ra, __fmul_rn(o.zs, rb));
    as = __fmaf_rn(as, ra, __fmul_rn(o.as, rb));
    ms = Ms;
    const float ta = ex2((mt - Mt) * kLog2e), tb = ex2((o.mt - Mt) * kLog2e);
    zt = __fmaf_rn(zt, ta, __fmul_rn(o.zt, tb));
    mt = Mt;
  }
};

// The accumulators of one thread while it sweeps its part of a row.  The exponent
// (x - max) * log2(e) is formed by one fused multiply-add, x * log2(e) - c with c =
// fl(max * log2(e)): the product is exact inside the fma, so the result differs from the
// exponent wanted only by the rounding of c, c_lo = max * log2(e) - c, which is the same for
// every element.  The sums therefore come out scaled by 2^c_lo exactly as they would with the
// difference taken first, and settle() takes the factor out (c_lo is given exactly by one more
// fma; |c_lo| < 1e-4, so 2^-c_lo = 1 - c_lo ln 2 to 1e-9).  The accuracy does not depend on the
// size of the logits.  When a maximum moves, the sums go from scale 2^-c_old to 2^-c_new by the
// factor 2^(c_old - c_new).  Student and teacher sums take the same steps, so a teacher equal
// to the student gives equal sums bit for bit.
struct RowSweep {
  float ms, cs, zs, as, mt, ct, zt;
  __device__ __forceinline__ void init() {
    ms = mt = cs = ct = kNegBig;
    zs = as = zt = 0.f;
  }
  // Fold N (s, t) pairs in; the maxima move only when a vector beats them.
  template <int N>
  __device__ __forceinline__ void add(const float (&s)[N], const float (&t)[N]) {
    const float vs = max_of<N>(s), vt = max_of<N>(t);
    if (vs > ms) {
      const float cn = vs * kLog2e, r = ex2(cs - cn);
      zs *= r;
      as *= r;
      ms = vs;
      cs = cn;
    }
    if (vt > mt) {
      const float cn = vt * kLog2e;
      zt *= ex2(ct - cn);
      mt = vt;
      ct = cn;
    }
#pragma unroll
    for (int i = 0; i < N; ++i) {
      const float es = ex2(fmaf(s[i], kLog2e, -cs));
      zs += es;
      as = fmaf(es, s[i] - t[i], as);
      zt += ex2(fmaf(t[i], kLog2e, -ct));
    }
  }
  __device__ __forceinline__ void add1(float s, float t) {
    const float a[1] = {s}, b[1] = {t};
    add<1>(a, b);
  }
  // The thread's partial on the scale of its own maxima, ready to be merged.
  __device__ __forceinline__ RowAcc settle() const {
    const float fs = -fmaf(ms, kLog2e, -cs) * kLn2, ft = -fmaf(mt, kLog2e, -ct) * kLn2;
    RowAcc r;
    r.ms = ms;
    r.zs = __fmaf_rn(zs, fs, zs);
    r.as = __fmaf_rn(as, fs, as);
    r.mt = mt;
    r.zt = __fmaf_rn(zt, ft, zt);
    return r;
  }
};

__device__ __forceinline__ RowAcc shfl_xor(const RowAcc &a, int lane_mask) {
  RowAcc o;
  o.ms = __shfl_xor_sync(0xffffffffu, a.ms, lane_mask);
  o.zs = __shfl_xor_sync(0xffffffffu, a.zs, lane_mask);
  o.as = __shfl_xor_sync(0xffffffffu, a.as, lane_mask);
  o.mt = __shfl_xor_sync(0xffffffffu, a.mt, lane_mask);
  o.zt = __shfl_xor_sync(0xffffffffu, a.zt, lane_mask);
  return o;
}

__device__ __forceinline__ RowAcc warp_reduce(RowAcc a) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) a.merge(shfl_xor(a, off));
  return a;
}

// Block-wide merge in a fixed order; the result is valid in every thread of
// warp 0.  scratch holds one RowAcc per warp.
template <int kThreads>
__device__ __forceinline__ RowAcc block_reduce(RowAcc a, RowAcc *scratch) {
  constexpr int kWarps = kThreads / 32;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  a = warp_reduce(a);
  if (lane == 0) scratch[warp] = a;
  __syncthreads();
  RowAcc r;
  r.init();
  if (warp == 0) {
    if (lane < kWarps) r = scratch[lane];
    r = warp_reduce(r);
  }
  return r;
}

// Per-row scalars derived from a finished RowAcc and the row's side inputs.
struct RowScalars {
  float lse_s, lse_t, kl, d;
};

}  // namespace fopd
