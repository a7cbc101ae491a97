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

// ------------------------------------------------------------------ the persistent-row skeleton
// The direct-load kernels run a fixed number of CTAs that draw row ids from a counter in the workspace
// header.  These pieces are the same in all of them.

// How one CTA of NT threads sees one row: geometry of the row image, this thread's share of the whole
// segments (s0, s0 + NT, ...: cnt of them), which thread does a ragged first / last segment element by
// element (thread 0 / thread 32), the label and whether the row takes part.
struct StreamRow {
  RowGeom g;
  int64_t row_off;   // first element of the row relative to the tensor (local row * pitch)
  int cnt, s0;
  bool edge_head, edge_tail, edge;
  int edge_seg;
  int y;
  bool valid;
};
template <typename T, int NT>
__device__ __forceinline__ StreamRow stream_row(int64_t local_row, long long global_row, int64_t row_stride, int64_t C,
                                                const int32_t* labels, const uint8_t* mask, int tid) {
  StreamRow w;
  w.g = row_geom<T>(local_row, row_stride, C);
  w.row_off = local_row * row_stride;
  const int n_int = w.g.seg_hi > w.g.seg_lo ? w.g.seg_hi - w.g.seg_lo : 0;   // segments wholly inside the row
  w.cnt = n_int > tid ? (n_int - tid + NT - 1) / NT : 0;
  w.s0 = w.g.seg_lo + tid;
  w.edge_head = (tid == 0) && w.g.seg_lo > 0;
  w.edge_tail = (tid == 32) && w.g.seg_hi < w.g.n_seg && (w.g.n_seg > 1 || w.g.seg_lo == 0);
  w.edge = w.edge_head || w.edge_tail;
  w.edge_seg = w.edge_head ? 0 : w.g.n_seg - 1;
  w.y = labels[global_row];
  w.valid = (mask == nullptr || mask[global_row] != 0) && w.y >= 0 && (int64_t)w.y < C;
  return w;
}

// The all-zero gradient row of a masked row: whole segments by 16-byte stores, ragged ones element by element.
template <typename T, int NT>
__device__ __forceinline__ void stream_zero_row(T* __restrict__ g_row, const StreamRow& w, int64_t C) {
  constexpr int V = SegOps<T>::V;
  uint4* g_img = reinterpret_cast<uint4*>(g_row - w.g.head);
  for (int i = 0; i < w.cnt; ++i) g_img[w.s0 + i * NT] = make_uint4(0u, 0u, 0u, 0u);
  if (w.edge) {
#pragma unroll
    for (int i = 0; i < V; ++i) {
      const int64_t c = (int64_t)w.edge_seg * V - w.g.head + i;
      if (c >= 0 && c < C) g_row[c] = Elem<T>::from_f32(0.f);
    }
  }
}

// Row ids: thread 0 draws the next id while the CTA works on the current one; two slots in shared memory
// alternate, and every row passes at least one __syncthreads() between the write and the reads of a slot.
__device__ __forceinline__ void stream_draw_row(long long* slot, WsHeader* hdr, long long row_begin, int tid) {
  if (tid == 0) *slot = row_begin + (long long)atomicAdd(&hdr->next_row, 1u);
}

// Called by every thread once the CTA's rows are written.  Returns true in the CTA that arrives last; that CTA has
// put the row counter back to zero for the next launch.  `flag` is one int of shared memory.
__device__ __forceinline__ bool stream_last_cta(WsHeader* hdr, int* flag, int tid) {
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const unsigned int prev = atomicAdd(&hdr->sched_done, 1u);
    *flag = (prev == gridDim.x - 1);
    if (*flag) { hdr->next_row = 0u; hdr->sched_done = 0u; __threadfence(); }
  }
  __syncthreads();
  return *flag != 0;
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
