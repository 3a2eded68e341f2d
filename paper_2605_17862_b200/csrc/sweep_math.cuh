// Per-vector arithmetic of the two sweeps of the on-chip kernel: the online
// max / sum-exp / KL accumulation of one 16-byte (student, teacher) vector pair
// and the gradient of one vector.  Two forms with identical results up to
// summation order: one fp32 lane per instruction, and two (sm_100a f32x2
// instructions: the sweeps are bound by instruction issue, and a packed
// instruction does the work of two for one issue slot).
#pragma once

#include "stream_kernels.cuh"

#ifndef FOPD_PACKED_MATH
#define FOPD_PACKED_MATH 0
#endif

namespace fopd {

// ------------------------------------------------------------------ two fp32 lanes per instruction
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float lo, float hi) {
  f32x2 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(f32x2 v, float &lo, float &hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
  f32x2 d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) {
  f32x2 d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ f32x2 sub2(f32x2 a, f32x2 b) {
  f32x2 d;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) {
  f32x2 d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ f32x2 ex2_2(f32x2 a) {
  float lo, hi;
  unpack2(a, lo, hi);
  return pack2(ex2(lo), ex2(hi));
}
// One 16-byte vector as fp32 pairs (adjacent logits share a pair).
template <int DT>
struct Pairs;
template <>
struct Pairs<FOPD_BF16> {
  static constexpr int kN = 4;
  __device__ static __forceinline__ void unpack(const uint4 &v, f32x2 (&x)[4]) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) x[i] = pack2(__uint_as_float(w[i] << 16), __uint_as_float(w[i] & 0xffff0000u));
  }
  __device__ static __forceinline__ uint4 pack(const f32x2 (&x)[4]) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float lo, hi;
      unpack2(x[i], lo, hi);
      __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
      w[i] = *reinterpret_cast<uint32_t *>(&h);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
  }
};
template <>
struct Pairs<FOPD_F32> {
  static constexpr int kN = 2;
  __device__ static __forceinline__ void unpack(const uint4 &v, f32x2 (&x)[2]) {
    x[0] = pack2(__uint_as_float(v.x), __uint_as_float(v.y));
    x[1] = pack2(__uint_as_float(v.z), __uint_as_float(v.w));
  }
  __device__ static __forceinline__ uint4 pack(const f32x2 (&x)[2]) {
    float a, b, c, d;
    unpack2(x[0], a, b);
    unpack2(x[1], c, d);
    return make_uint4(__float_as_uint(a), __float_as_uint(b), __float_as_uint(c), __float_as_uint(d));
  }
};
template <int N>
__device__ __forceinline__ float max_of_pairs(const f32x2 (&x)[N]) {
  float v[2 * N];
#pragma unroll
  for (int i = 0; i < N; ++i) unpack2(x[i], v[2 * i], v[2 * i + 1]);
  if (N == 4) return fmaxf(max3(v[0], v[1], v[2]), max3(v[3], v[4], max3(v[5], v[6], v[7])));
  return fmaxf(fmaxf(v[0], v[1]), fmaxf(v[2 * N - 2], v[2 * N - 1]));
}

#if FOPD_PACKED_MATH
// Online accumulators of one thread with the sums kept as fp32 pairs (even / odd logits).
// Student and teacher sums go through the same operations in the same order.
template <int DT>
struct SweepAcc {
  float ms, mt;
  f32x2 zs, as, zt;
  __device__ __forceinline__ void init() {
    ms = mt = kNegBig;
    zs = as = zt = pack2(0.f, 0.f);
  }
  __device__ __forceinline__ void rescale(float vs, float vt) {
    if (vs > ms) {
      const float r = ex2((ms - vs) * kLog2e);
      const f32x2 r2 = pack2(r, r);
      zs = mul2(zs, r2);
      as = mul2(as, r2);
      ms = vs;
    }
    if (vt > mt) {
      const float r = ex2((mt - vt) * kLog2e);
      zt = mul2(zt, pack2(r, r));
      mt = vt;
    }
  }
  __device__ __forceinline__ void add(const uint4 &sv, const uint4 &tv) {
    constexpr int N = Pairs<DT>::kN;
    f32x2 s[N], t[N];
    Pairs<DT>::unpack(sv, s);
    Pairs<DT>::unpack(tv, t);
    rescale(max_of_pairs<N>(s), max_of_pairs<N>(t));
    const float bs = -ms * kLog2e, bt = -mt * kLog2e;
    const f32x2 L = pack2(kLog2e, kLog2e), bs2 = pack2(bs, bs), bt2 = pack2(bt, bt);
#pragma unroll
    for (int i = 0; i < N; ++i) {
      const f32x2 es = ex2_2(fma2(s[i], L, bs2));
      const f32x2 et = ex2_2(fma2(t[i], L, bt2));
      zs = add2(zs, es);
      zt = add2(zt, et);
      as = fma2(es, sub2(s[i], t[i]), as);
    }
  }
  // one more logit pair (scalar tail of a row): goes to the low lanes
  __device__ __forceinline__ void add1(float s, float t) {
    rescale(s, t);
    const float es = ex2((s - ms) * kLog2e), et = ex2((t - mt) * kLog2e);
    zs = add2(zs, pack2(es, 0.f));
    zt = add2(zt, pack2(et, 0.f));
    as = fma2(pack2(es, 0.f), pack2(s - t, 0.f), as);
  }
  __device__ __forceinline__ RowAcc fold() const {
    RowAcc r;
    float a, b;
    r.ms = ms;
    r.mt = mt;
    unpack2(zs, a, b);
    r.zs = a + b;
    unpack2(as, a, b);
    r.as = a + b;
    unpack2(zt, a, b);
    r.zt = a + b;
    return r;
  }
};

// Gradient of one vector (see GradRow) without the stored token's extra term.
template <int DT>
__device__ __forceinline__ uint4 grad_body(const uint4 &sv, const uint4 &tv, const GradRow &r) {
  constexpr int N = Pairs<DT>::kN;
  f32x2 s[N], t[N], o[N];
  Pairs<DT>::unpack(sv, s);
  Pairs<DT>::unpack(tv, t);
  const f32x2 L = pack2(kLog2e, kLog2e), e0 = pack2(r.e0, r.e0), K = pack2(r.K, r.K);
#pragma unroll
  for (int i = 0; i < N; ++i) o[i] = mul2(ex2_2(fma2(s[i], L, e0)), sub2(sub2(s[i], t[i]), K));
  return Pairs<DT>::pack(o);
}
#else
template <int DT>
struct SweepAcc {
  RowAcc acc;
  __device__ __forceinline__ void init() { acc.init(); }
  __device__ __forceinline__ void add(const uint4 &sv, const uint4 &tv) {
    constexpr int P = Elem<DT>::kPerVec;
    float s[P], t[P];
    Elem<DT>::unpack(sv, s);
    Elem<DT>::unpack(tv, t);
    acc.add<P>(s, t);
  }
  __device__ __forceinline__ void add1(float s, float t) { acc.add1(s, t); }
  __device__ __forceinline__ RowAcc fold() const { return acc; }
};

template <int DT>
__device__ __forceinline__ uint4 grad_body(const uint4 &sv, const uint4 &tv, const GradRow &r) {
  using E = Elem<DT>;
  constexpr int P = E::kPerVec;
  float s[P], t[P], o[P];
  E::unpack(sv, s);
  E::unpack(tv, t);
#pragma unroll
  for (int i = 0; i < P; ++i) o[i] = ex2(fmaf(s[i], kLog2e, r.e0)) * ((s[i] - t[i]) - r.K);
  return E::pack(o);
}
#endif

}  // namespace fopd
