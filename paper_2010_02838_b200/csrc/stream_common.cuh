// Shared pieces of the direct-load ("stream") row kernels: launch shape, per-CTA shared memory,
// cache-policy loads and stores, scalar look-ups in a row.
#pragma once
#include "common.cuh"
#include "seg_math.cuh"

#ifndef STREAM_HINTS
#define STREAM_HINTS 5   // bit 0: own-row loads of pass A ask L2 to keep the lines; bit 1: peer loads, bit 2: gradient stores marked evict-first
#endif

namespace codistill {

// Launch shape by peer count (measured on B200): up to three peers 256 threads x 3 CTAs per SM
// (80 registers, two own segments and their peer segments in flight per thread); more peers 128
// threads x 4 CTAs (128 registers), one own segment and all its peer segments in flight.
constexpr int kStreamMaxWarps = 8;
constexpr int kStreamMaxPeers = 7;
constexpr int kBatchA = 4;   // segments per thread in flight in pass A
constexpr int kBatchB = 2;   // own segments per thread in flight in pass B with few peers
__host__ __device__ constexpr int stream_threads(int peers) { return peers >= 4 ? 128 : 256; }
__host__ __device__ constexpr int stream_ctas_per_sm(int peers) { return peers >= 4 ? 4 : 3; }

struct StreamShared {
  float4 red[2][kStreamMaxWarps];                              // pass-A partials, alternating between rows
  float endred[2][kStreamMaxWarps * (1 + 3 * kStreamMaxPeers)];  // pass-B partials, alternating between rows
  float cen[2][kStreamMaxPeers][kStreamMaxWarps];               // centred distance: per-peer class sums, alternating between rows
  long long next_row[2];
  double fin[32];
  int last_flag;
};

// 16-byte global load / store with an L2 eviction policy (see make_policy_*).
// Batches of a thread's segments requested from the L2 ahead of their loads (0: none): the own row in the
// statistics pass, the peers in the gradient pass.  One batch ahead in both is 10 % faster with one peer
// (few independent loads in flight per thread); with seven peers it changes nothing or costs 2 %, and two
// batches ahead were slower everywhere.
__host__ __device__ constexpr int stream_ahead(int peers) { return peers <= 3 ? 1 : 0; }
__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

__device__ __forceinline__ uint4 ldg_policy(const uint4* p, uint64_t pol) {
  uint4 r;
  asm volatile("ld.global.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p), "l"(pol));
  return r;
}
__device__ __forceinline__ void stg_policy(uint4* p, const uint4& v, uint64_t pol) {
  asm volatile("st.global.L2::cache_hint.v4.u32 [%0], {%1,%2,%3,%4}, %5;" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w), "l"(pol) : "memory");
}
__device__ __forceinline__ uint64_t make_policy_keep() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ uint64_t make_policy_stream() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}

// First column of segment `s` of the row image whose value equals m, or INT_MAX; reads single elements.
template <typename T>
__device__ __noinline__ int first_equal_global(const T* __restrict__ z_row, int s, int head, int64_t C, float m) {
  constexpr int V = SegOps<T>::V;
  int first = 0x7fffffff;
#pragma unroll
  for (int i = V - 1; i >= 0; --i) {
    const int64_t c = (int64_t)s * V - head + i;
    if (c >= 0 && c < C && Elem<T>::to_f32(z_row[c]) == m) first = (int)c;
  }
  return first;
}

}  // namespace codistill
