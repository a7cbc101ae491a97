// Arithmetic on 16-byte segments of a logit row, shared by the row kernels: unpacking to packed
// fp32 pairs, running maxima, the shifted exponential, order-preserving keys for integer warp
// reductions and the geometry of a row image (the 16-byte aligned byte range that holds a row).
#pragma once
#include "common.cuh"

namespace codistill {

// ------------------------------------------------------------------ 16-byte segments
template <typename T> struct SegOps;
template <> struct SegOps<float> {
  static constexpr int V = 4;   // elements per segment
  static constexpr int H = 2;   // float2 pairs per segment
  using macc = float;           // running-maximum accumulator
  __device__ static void unpack(const uint4& r, float (&o)[4]) {
    o[0] = __uint_as_float(r.x); o[1] = __uint_as_float(r.y); o[2] = __uint_as_float(r.z); o[3] = __uint_as_float(r.w);
  }
  __device__ static void unpack2(const uint4& r, float2 (&o)[2]) {
    o[0] = make_float2(__uint_as_float(r.x), __uint_as_float(r.y));
    o[1] = make_float2(__uint_as_float(r.z), __uint_as_float(r.w));
  }
  __device__ static uint4 pack2(const float2 (&v)[2]) {
    return make_uint4(__float_as_uint(v[0].x), __float_as_uint(v[0].y), __float_as_uint(v[1].x), __float_as_uint(v[1].y));
  }
  __device__ static macc neg_inf() { return -INFINITY; }
  __device__ static macc fold(const uint4& r) {
    return fmaxf(fmaxf(__uint_as_float(r.x), __uint_as_float(r.y)), fmaxf(__uint_as_float(r.z), __uint_as_float(r.w)));
  }
  __device__ static macc mmax(macc a, macc b) { return fmaxf(a, b); }
  __device__ static macc from_scalar(float v) { return v; }
  __device__ static float to_float(macc a) { return a; }
};
template <> struct SegOps<__nv_bfloat16> {
  static constexpr int V = 8;
  static constexpr int H = 4;
  using macc = __nv_bfloat162;  // two running maxima (even / odd columns), folded at the end
  __device__ static void unpack(const uint4& r, float (&o)[8]) {
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      o[2 * i] = __uint_as_float(w[i] << 16);
      o[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
  }
  __device__ static void unpack2(const uint4& r, float2 (&o)[4]) {
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) o[i] = make_float2(__uint_as_float(w[i] << 16), __uint_as_float(w[i] & 0xFFFF0000u));
  }
  __device__ static uint4 pack2(const float2 (&v)[4]) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const __nv_bfloat162 p = __floats2bfloat162_rn(v[i].x, v[i].y);
      w[i] = *reinterpret_cast<const uint32_t*>(&p);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
  }
  __device__ static macc neg_inf() { return __floats2bfloat162_rn(-INFINITY, -INFINITY); }
  __device__ static macc fold(const uint4& r) {
    const __nv_bfloat162 a = __hmax2(*reinterpret_cast<const __nv_bfloat162*>(&r.x), *reinterpret_cast<const __nv_bfloat162*>(&r.y));
    const __nv_bfloat162 b = __hmax2(*reinterpret_cast<const __nv_bfloat162*>(&r.z), *reinterpret_cast<const __nv_bfloat162*>(&r.w));
    return __hmax2(a, b);
  }
  __device__ static macc mmax(macc a, macc b) { return __hmax2(a, b); }
  __device__ static macc from_scalar(float v) { return __floats2bfloat162_rn(v, v); }  // v is a bf16 value: exact
  __device__ static float to_float(macc a) { return fmaxf(__low2float(a), __high2float(a)); }
};

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// exp(z - m) for a pair of columns.  fp32 logits keep full precision (their gradient tolerance is
// 1e-6 absolute); bf16 logits fold the shift into one packed FMA feeding the hardware exp2.
template <typename T>
__device__ __forceinline__ float2 exp_shift2(float2 z, float m, float2 l2e, float2 neg_m_l2e) {
  if constexpr (sizeof(T) == 4) {
    return make_float2(expf(z.x - m), expf(z.y - m));
  } else {
    const float2 t = __ffma2_rn(z, l2e, neg_m_l2e);
    return make_float2(ex2_approx(t.x), ex2_approx(t.y));
  }
}

// 2^x for the rescaling factors of the online softmax: exact enough for the 1e-6 gradient tolerance of
// fp32 logits, the bare hardware instruction for bf16 logits.
template <typename T>
__device__ __forceinline__ float rescale_exp2(float x) {
  if constexpr (sizeof(T) == 4) return exp2f(x); else return ex2_approx(x);
}

// Order-preserving map between floats and unsigned integers (for integer warp reductions).
__device__ __forceinline__ unsigned float_order_key(float f) {
  const unsigned u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float float_from_order_key(unsigned k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// Warp maximum through one integer reduction on the order-preserving key.
__device__ __forceinline__ float warp_max_redux(float v) {
  return float_from_order_key(__reduce_max_sync(0xffffffffu, float_order_key(v)));
}

// Geometry of one row image.
struct RowGeom {
  int head;      // elements of the first segment that precede the row
  int n_seg;     // 16-byte segments of the image
  int seg_lo;    // first segment that lies wholly inside the row
  int seg_hi;    // one past the last such segment
};
template <typename T>
__device__ __forceinline__ RowGeom row_geom(int64_t local_row, int64_t row_stride, int64_t classes) {
  constexpr int V = SegOps<T>::V;
  RowGeom g;
  g.head = (int)((local_row * row_stride) & (V - 1));
  const int64_t end = g.head + classes;  // in elements, from the image start
  g.n_seg = (int)((end + V - 1) / V);
  g.seg_lo = g.head ? 1 : 0;
  g.seg_hi = (end & (V - 1)) ? g.n_seg - 1 : g.n_seg;
  return g;
}

// Geometry shared by every row of a call: segments of the longest row image.
template <typename T>
__host__ __device__ inline int64_t max_row_segments(int64_t row_stride, int64_t classes) {
  constexpr int V = 16 / (int)sizeof(T);
  const int64_t head_max = (row_stride % V == 0) ? 0 : V - 1;
  return (head_max + classes + V - 1) / V;
}

}  // namespace codistill
