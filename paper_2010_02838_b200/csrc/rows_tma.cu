// Persistent, warp-specialised kernel for long rows ("tma" regime), MSE-on-logits distance.
//
// One CTA per SM.  Warp 0 is the producer: it draws row ids from a global counter and moves row
// images from HBM into shared memory with 1-D bulk asynchronous copies (cp.async.bulk) that
// complete on mbarriers.  The own row of a model stays resident in one of one or two row
// buffers; the n-1 peer rows are streamed chunk by chunk (chunk-major: chunk k of peer 0, 1, ...,
// then chunk k+1) through a ring of 16 KiB stages.  The 16 consumer warps make one pass over the
// resident own row for the softmax statistics, then consume the ring: per 16-byte segment they
// accumulate sum_j (z - z_j) and sum_j (z - z_j)^2, track what the arg-max agreement needs, and
// write the gradient with 128-bit stores.  Every logit is read from HBM exactly once and the
// gradient is written once.
//
// A "row image" is the 16-byte aligned byte range that contains the row: rows whose byte length
// is not a multiple of 16 start at varying offsets `head` inside their first segment.  Segments
// that are only partly inside the row ("edge" segments) take a masked slow path.
#include "common.cuh"

namespace codistill {

// Tuning constants (overridable at compile time for experiments).
#ifndef CODISTILL_TMA_CONSUMER_WARPS
#define CODISTILL_TMA_CONSUMER_WARPS 16
#endif
#ifndef CODISTILL_TMA_CTAS_PER_SM
#define CODISTILL_TMA_CTAS_PER_SM 1
#endif
#ifndef CODISTILL_TMA_CHUNK_BYTES
#define CODISTILL_TMA_CHUNK_BYTES 16384
#endif
constexpr int kConsumerWarps = CODISTILL_TMA_CONSUMER_WARPS;
constexpr int kCtasPerSm = CODISTILL_TMA_CTAS_PER_SM;
constexpr int kConsumers = kConsumerWarps * 32;
constexpr int kTmaThreads = kConsumers + 32;
constexpr int kChunkBytes = CODISTILL_TMA_CHUNK_BYTES;
constexpr int kSegPerChunk = kChunkBytes / 16;
constexpr int kSegPerThread = kSegPerChunk / kConsumers;
static_assert(kSegPerThread * kConsumers == kSegPerChunk, "a chunk splits evenly over the consumer threads");
constexpr int kMaxStages = 12;
constexpr int kCtrlBytes = 4096;
constexpr int kOwnPieceBytes = 32768;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;  // bounded waits: 2 s, then CODISTILL_DEV_TIMEOUT

struct TmaCfg {
  int own_bufs;
  int stages;
  uint32_t own_buf_bytes;
  uint32_t smem_bytes;
};

struct RowInfo {
  long long row;  // global row id, -1 = no more rows
  int valid;
  int label;
};

struct Ctrl {  // lives at the start of dynamic shared memory
  uint64_t own_full[2];
  uint64_t own_empty[2];
  uint64_t ring_full[kMaxStages];
  uint64_t ring_empty[kMaxStages];
  RowInfo info[2];
  int abort_flag;
  int last_flag;
  float red[2][kConsumerWarps * 24];  // reduction scratch of the consumers, two alternating halves
  double fin[32];
};
static_assert(sizeof(Ctrl) <= kCtrlBytes, "control block fits its slot");

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// global -> shared bulk copy (no multicast); dst, src and bytes are multiples of 16
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ unsigned long long global_timer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void consumer_bar() { asm volatile("bar.sync 1, %0;" ::"n"(kConsumers) : "memory"); }

// Wait for a phase of an mbarrier, but never for ever: after kWaitLimitNs the CTA-wide abort flag
// and the device status are set and every later wait returns at once (results are then invalid).
__device__ __forceinline__ void wait_bounded(uint64_t* bar, uint32_t parity, Ctrl* ctrl, WsHeader* hdr) {
  if (mbar_try_wait(bar, parity)) return;
  volatile int* abort_flag = &ctrl->abort_flag;
  uint32_t polls = 0;
  unsigned long long t0 = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++polls & 0x3FFu) == 0) {
      if (*abort_flag) return;
      const unsigned long long now = global_timer_ns();
      if (t0 == 0) {
        t0 = now;
      } else if (now - t0 > kWaitLimitNs) {
        *abort_flag = 1;
        atomicOr(&hdr->status, CODISTILL_DEV_TIMEOUT);
        return;
      }
    }
  }
}

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

// Block reductions among the 512 consumer threads (one named barrier each).
struct ConsumerReduce {
  Ctrl* ctrl;
  int toggle;
  int warp, lane;  // consumer warp index 0..15
  template <int N>
  __device__ __forceinline__ void sum(float (&v)[N]) {
    float* s = ctrl->red[toggle];
#pragma unroll
    for (int k = 0; k < N; ++k) {
      v[k] = warp_sum(v[k]);
      if (lane == 0) s[k * kConsumerWarps + warp] = v[k];
    }
    consumer_bar();
#pragma unroll
    for (int k = 0; k < N; ++k) v[k] = warp_sum(lane < kConsumerWarps ? s[k * kConsumerWarps + lane] : 0.f);
    toggle ^= 1;
  }
  template <int N>
  __device__ __forceinline__ void max(float (&v)[N]) {
    float* s = ctrl->red[toggle];
#pragma unroll
    for (int k = 0; k < N; ++k) {
      v[k] = warp_max(v[k]);
      if (lane == 0) s[k * kConsumerWarps + warp] = v[k];
    }
    consumer_bar();
#pragma unroll
    for (int k = 0; k < N; ++k) v[k] = warp_max(lane < kConsumerWarps ? s[k * kConsumerWarps + lane] : -INFINITY);
    toggle ^= 1;
  }
  __device__ __forceinline__ int min_int(int v) {
    int* s = reinterpret_cast<int*>(ctrl->red[toggle]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = ::min(v, __shfl_xor_sync(0xffffffffu, v, o));
    if (lane == 0) s[warp] = v;
    consumer_bar();
    v = lane < kConsumerWarps ? s[lane] : 0x7fffffff;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = ::min(v, __shfl_xor_sync(0xffffffffu, v, o));
    toggle ^= 1;
    return v;
  }
};

// ------------------------------------------------------------------ producer helpers
// Moves `img_bytes` of a row image from `src` (16-byte aligned) to `dst`, completing on `bar`.
// `tma_bytes` <= img_bytes is the part that may be read as whole segments; the elements between
// tma_bytes and valid_end (a partial last segment at the very end of a tensor) are fetched with
// plain loads by the lanes of the producer warp.  Called by the whole producer warp.
template <typename T>
__device__ __forceinline__ void produce_copy(char* dst, const char* src, uint32_t begin, uint32_t end, uint32_t tma_limit,
                                             uint32_t valid_end, uint64_t* bar, int lane) {
  // [begin, end) is the byte range of the image handled by this copy
  const uint32_t tma_end = end < tma_limit ? end : tma_limit;
  if (end > tma_limit) {  // partial last segment that must not be read as a whole
    const uint32_t first = tma_limit > begin ? tma_limit : begin;
    const uint32_t off = first + (uint32_t)lane * (uint32_t)sizeof(T);
    if (off < valid_end) *reinterpret_cast<T*>(dst + (off - begin)) = *reinterpret_cast<const T*>(src + off);
    __syncwarp();
  }
  if (lane == 0) {
    const uint32_t bytes = tma_end > begin ? tma_end - begin : 0u;
    mbar_arrive_expect_tx(bar, bytes);
    for (uint32_t o = 0; o < bytes; o += kOwnPieceBytes) {
      const uint32_t piece = bytes - o < (uint32_t)kOwnPieceBytes ? bytes - o : (uint32_t)kOwnPieceBytes;
      bulk_g2s(dst + o, src + begin + o, piece, bar);
    }
  }
}

// First column of segment `s` whose value equals m, or INT_MAX.
template <typename T>
__device__ __forceinline__ int first_equal(const char* img, int s, int head, int64_t C, float m) {
  constexpr int V = SegOps<T>::V;
  float z[V];
  SegOps<T>::unpack(*reinterpret_cast<const uint4*>(img + (size_t)s * 16), z);
  int first = 0x7fffffff;
#pragma unroll
  for (int i = V - 1; i >= 0; --i) {
    const int64_t c = (int64_t)s * V - head + i;
    if (c >= 0 && c < C && z[i] == m) first = (int)c;
  }
  return first;
}

// Element-by-element treatment of one peer segment that is ragged (partly outside the row) or holds
// the own arg-max column: differences z - v with zeros outside the row, and the maxima of the
// peer's values before / after / at column a_own (a_own < 0: not wanted).
template <typename T>
struct SlowPeer {
  float2 d2[SegOps<T>::H];
  float lt, ge, za;
};
template <typename T>
struct SegPairs {  // one segment as float2 pairs, passed by value so that the caller's copy stays in registers
  float2 v[SegOps<T>::H];
};
template <typename T>
__device__ __noinline__ SlowPeer<T> slow_peer(SegPairs<T> zs, uint4 raw, int seg, int head, int64_t C, int a_own) {
  constexpr int V = SegOps<T>::V;
  const float2 (&z2)[SegOps<T>::H] = zs.v;
  float v[V];
  SegOps<T>::unpack(raw, v);
  SlowPeer<T> o;
  o.lt = -INFINITY; o.ge = -INFINITY; o.za = -INFINITY;
#pragma unroll
  for (int i = 0; i < V; ++i) {
    const int64_t c = (int64_t)seg * V - head + i;
    const bool in = c >= 0 && c < C;
    const float z = (i & 1) ? z2[i >> 1].y : z2[i >> 1].x;
    const float d = in ? z - v[i] : 0.f;
    if (i & 1) o.d2[i >> 1].y = d; else o.d2[i >> 1].x = d;
    if (in && a_own >= 0) {
      if (c < a_own) o.lt = fmaxf(o.lt, v[i]);
      else if (c > a_own) o.ge = fmaxf(o.ge, v[i]);
      else o.za = v[i];
    }
  }
  return o;
}

// ------------------------------------------------------------------ the kernel
template <typename T, int P, bool PW>
__global__ void __launch_bounds__(kTmaThreads, kCtasPerSm) rows_tma_kernel(const __grid_constant__ KArgs a, const TmaCfg cfg) {
  constexpr int V = SegOps<T>::V;
  constexpr int H = SegOps<T>::H;
  constexpr int PD = P > 0 ? P : 1;
  constexpr int ES = (int)sizeof(T);
  extern __shared__ __align__(128) unsigned char smem_raw[];
  Ctrl* ctrl = reinterpret_cast<Ctrl*>(smem_raw);
  char* own_base = reinterpret_cast<char*>(smem_raw) + kCtrlBytes;
  char* ring_base = own_base + (size_t)cfg.own_bufs * cfg.own_buf_bytes;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_own = cfg.own_bufs, n_stage = cfg.stages;
  const int64_t C = a.classes;
  const bool with_term = (P >= 1 && a.alpha != 0.f);
  const bool stream_peers = (P >= 1) && (with_term || a.want_flags);

  if (threadIdx.x == 0) {
    for (int b = 0; b < 2; ++b) { mbar_init(&ctrl->own_full[b], 1); mbar_init(&ctrl->own_empty[b], kConsumerWarps); }
    for (int s = 0; s < kMaxStages; ++s) { mbar_init(&ctrl->ring_full[s], 1); mbar_init(&ctrl->ring_empty[s], kConsumerWarps); }
    ctrl->abort_flag = 0;
    ctrl->last_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  if (warp == 0) {
    // ============================== producer warp ==============================
    uint32_t q = 0;  // ring items issued so far
    int last_it[2] = {-1, -1};
    // Row ids come from a global counter.  The counter and the row's mask byte and label are fetched
    // two and one iterations ahead (lane 0), so that their latency never sits between two rows.
    long long t_next = 0, t_next2 = 0;
    int mask_next = 0, label_next = 0;
    if (lane == 0) {
      t_next = a.row_begin + (long long)atomicAdd(&a.hdr->next_row, 1u);
      t_next2 = a.row_begin + (long long)atomicAdd(&a.hdr->next_row, 1u);
      if (t_next < a.row_end) { mask_next = a.mask ? a.mask[t_next] : 1; label_next = a.labels[t_next]; }
    }
    for (int it = 0;; ++it) {
      long long r = t_next;
      int mask_v = mask_next, label_v = label_next;
      if (lane == 0) {
        t_next = t_next2;
        t_next2 = a.row_begin + (long long)atomicAdd(&a.hdr->next_row, 1u);
        if (t_next < a.row_end) { mask_next = a.mask ? a.mask[t_next] : 1; label_next = a.labels[t_next]; }
      }
      r = __shfl_sync(0xffffffffu, r, 0);
      mask_v = __shfl_sync(0xffffffffu, mask_v, 0);
      label_v = __shfl_sync(0xffffffffu, label_v, 0);
      const int b = it % n_own;
      const bool more = r < a.row_end;
      const bool valid = more && mask_v != 0 && label_v >= 0 && (int64_t)label_v < C;
      const int64_t lr = r - a.row_begin;
      const RowGeom g = row_geom<T>(valid ? lr : 0, a.row_stride, C);
      const uint32_t img_bytes = (uint32_t)g.n_seg * 16u;
      const uint32_t valid_end = (uint32_t)(g.head + C) * ES;
      // The last row of the whole call may end inside a segment that reaches past the tensor.
      const bool clip = (r == a.rows_total - 1) && ((a.row_stride - C) * ES < 16) && (valid_end & 15u);
      const uint32_t tma_limit = clip ? (valid_end & ~15u) : img_bytes;
      const int64_t row_off = lr * a.row_stride * ES - (int64_t)g.head * ES;  // image start relative to the tensor
      const int n_items = (valid && stream_peers) ? ((g.n_seg + kSegPerChunk - 1) / kSegPerChunk) * P : 0;
      auto issue_item = [&](int idx) {
        const int k = idx / PD, j = idx - k * PD;
        const uint32_t begin = (uint32_t)k * kChunkBytes;
        const uint32_t end = begin + kChunkBytes < img_bytes ? begin + kChunkBytes : img_bytes;
        const int s = q % n_stage;
        if (q >= (uint32_t)n_stage) wait_bounded(&ctrl->ring_empty[s], ((q / n_stage) - 1) & 1, ctrl, a.hdr);
        produce_copy<T>(ring_base + (size_t)s * kChunkBytes, reinterpret_cast<const char*>(a.peers[j]) + row_off, begin, end,
                        tma_limit, valid_end, &ctrl->ring_full[s], lane);
        ++q;
      };
      // With a single row buffer the next own row cannot be fetched before the current row is
      // finished; fill the ring with the next row's first peer chunks meanwhile.  Never more than
      // the ring holds, or the producer would wait for stages the consumers cannot yet free.
      const int pre = (n_own == 1) ? (n_items < n_stage ? n_items : n_stage) : 0;
      for (int idx = 0; idx < pre; ++idx) issue_item(idx);
      if (it >= n_own) wait_bounded(&ctrl->own_empty[b], ((it / n_own) - 1) & 1, ctrl, a.hdr);
      last_it[b] = it;
      if (lane == 0) {
        ctrl->info[b].row = more ? r : -1;
        ctrl->info[b].valid = valid;
        ctrl->info[b].label = label_v;
      }
      if (!valid) {
        __syncwarp();
        if (lane == 0) mbar_arrive(&ctrl->own_full[b]);
        if (!more) break;
        continue;
      }
      produce_copy<T>(own_base + (size_t)b * cfg.own_buf_bytes, reinterpret_cast<const char*>(a.own) + row_off, 0u, img_bytes,
                      tma_limit, valid_end, &ctrl->own_full[b], lane);
      for (int idx = pre; idx < n_items; ++idx) issue_item(idx);
    }
    // Before leaving, make sure no copy armed by this warp is still in flight (bounded).
    for (int b = 0; b < n_own; ++b)
      if (last_it[b] >= 0) wait_bounded(&ctrl->own_full[b], (last_it[b] / n_own) & 1, ctrl, a.hdr);
    for (uint32_t i = 0; i < (uint32_t)n_stage && i < q; ++i) {
      const uint32_t qi = q - 1 - i;
      wait_bounded(&ctrl->ring_full[qi % n_stage], (qi / n_stage) & 1, ctrl, a.hdr);
    }
  } else {
    // ============================== consumer warps ==============================
    const int tid = threadIdx.x - 32;
    ConsumerReduce red{ctrl, 0, warp - 1, lane};
    float w = 1.f;
    if (a.reduction == CODISTILL_REDUCE_MEAN_VALID) {
      const int64_t nv = total_valid(a);
      w = 1.f / (float)(nv > 1 ? nv : 1);
    }
    const float inv_P = P >= 1 ? 1.f / (float)P : 0.f;
    uint32_t q = 0;
    for (int it = 0;; ++it) {
      const int b = it % n_own;
      wait_bounded(&ctrl->own_full[b], (it / n_own) & 1, ctrl, a.hdr);
      const long long r = ctrl->info[b].row;
      if (r < 0) break;
      const bool valid = ctrl->info[b].valid != 0;
      const int y = ctrl->info[b].label;
      const int64_t lr = r - a.row_begin;
      const RowGeom g = row_geom<T>(lr, a.row_stride, C);
      const char* img = own_base + (size_t)b * cfg.own_buf_bytes;
      char* g_img = a.grad ? reinterpret_cast<char*>(a.grad) + lr * a.row_stride * ES - (int64_t)g.head * ES : nullptr;

      if (!valid) {
        if (g_img) {
          for (int s = tid; s < g.n_seg; s += kConsumers) {
            if (s >= g.seg_lo && s < g.seg_hi) {
              *reinterpret_cast<uint4*>(g_img + (size_t)s * 16) = make_uint4(0u, 0u, 0u, 0u);
            } else {
#pragma unroll
              for (int i = 0; i < V; ++i) {
                const int64_t c = (int64_t)s * V - g.head + i;
                if (c >= 0 && c < C) reinterpret_cast<T*>(g_img + (size_t)s * 16)[i] = Elem<T>::from_f32(0.f);
              }
            }
          }
        }
        if (tid == 0) { a.row_loss[r] = 0.f; a.row_flags[r] = 0u; }
        __syncwarp();
        if (lane == 0) mbar_arrive(&ctrl->own_empty[b]);
        continue;
      }

      // ---------------- pass over the resident own row: max, then sum exp / sum z
      // Interior segments take the packed path; the (at most two) ragged edge segments are handled
      // element by element by one thread each.
      const int e0 = g.seg_lo > 0 ? 0 : -1;
      const int e1 = (g.seg_hi < g.n_seg && !(e0 == 0 && g.n_seg == 1)) ? g.n_seg - 1 : -1;
      const int my_edge = (tid == 0) ? e0 : (tid == 32 ? e1 : -1);
      typename SegOps<T>::macc mx = SegOps<T>::neg_inf();
      for (int s = g.seg_lo + tid; s < g.seg_hi; s += kConsumers)
        mx = SegOps<T>::mmax(mx, SegOps<T>::fold(*reinterpret_cast<const uint4*>(img + (size_t)s * 16)));
      float m_t = SegOps<T>::to_float(mx);
      if (my_edge >= 0) {
        float z[V];
        SegOps<T>::unpack(*reinterpret_cast<const uint4*>(img + (size_t)my_edge * 16), z);
#pragma unroll
        for (int i = 0; i < V; ++i) {
          const int64_t c = (int64_t)my_edge * V - g.head + i;
          if (c >= 0 && c < C) m_t = fmaxf(m_t, z[i]);
        }
      }
      float mm[1] = {m_t};
      red.max(mm);
      const float m = mm[0];
      const float2 l2e2 = make_float2(kLog2e, kLog2e);
      const float2 nml2 = make_float2(-m * kLog2e, -m * kLog2e);
      float2 s2[H], zs2[H];
#pragma unroll
      for (int i = 0; i < H; ++i) { s2[i] = make_float2(0.f, 0.f); zs2[i] = make_float2(0.f, 0.f); }
      for (int s = g.seg_lo + tid; s < g.seg_hi; s += kConsumers) {
        float2 z2[H];
        SegOps<T>::unpack2(*reinterpret_cast<const uint4*>(img + (size_t)s * 16), z2);
#pragma unroll
        for (int i = 0; i < H; ++i) {
          s2[i] = __fadd2_rn(s2[i], exp_shift2<T>(z2[i], m, l2e2, nml2));
          zs2[i] = __fadd2_rn(zs2[i], z2[i]);
        }
      }
      float acc[2] = {0.f, 0.f};
#pragma unroll
      for (int i = 0; i < H; ++i) { acc[0] += s2[i].x + s2[i].y; acc[1] += zs2[i].x + zs2[i].y; }
      if (my_edge >= 0) {
        float z[V];
        SegOps<T>::unpack(*reinterpret_cast<const uint4*>(img + (size_t)my_edge * 16), z);
#pragma unroll
        for (int i = 0; i < V; ++i) {
          const int64_t c = (int64_t)my_edge * V - g.head + i;
          if (c >= 0 && c < C) {
            const float2 e = exp_shift2<T>(make_float2(z[i], z[i]), m, l2e2, nml2);
            acc[0] += e.x;
            acc[1] += z[i];
          }
        }
      }
      red.sum(acc);
      const float S = acc[0], sum_z = acc[1];
      const float zy = Elem<T>::to_f32(reinterpret_cast<const T*>(img)[g.head + y]);
      const float ce = (m + logf(S)) - (1.f - a.eps) * zy - (a.eps / (float)C) * sum_z;

      // ---------------- first arg-max of the own row (only threads that hold the maximum rescan)
      int a_own = 0;
      if (a.want_flags) {
        int first = 0x7fffffff;
        if (m_t == m) {
          if (my_edge == e0 && e0 >= 0) first = first_equal<T>(img, e0, g.head, C, m);
          for (int s = g.seg_lo + tid; s < g.seg_hi && first == 0x7fffffff; s += kConsumers)
            first = first_equal<T>(img, s, g.head, C, m);
          if (first == 0x7fffffff && my_edge == e1 && e1 >= 0) first = first_equal<T>(img, e1, g.head, C, m);
        }
        a_own = red.min_int(first);
      }
      const int seg_a = a.want_flags ? (g.head + a_own) / V : -1;

      // ---------------- stream the peers chunk by chunk, write the gradient
      const float cp = w / S;                                                     // e_c -> w * p_c
      const float cd = with_term ? w * a.alpha * (2.f / (float)C) * inv_P : 0.f;  // sum_j d -> w * alpha * dD
      const float cq = w * a.eps / (float)C;
      const float cy = w * (1.f - a.eps);
      const float2 cp2 = make_float2(cp, cp), cd2 = make_float2(cd, cd), ncq2 = make_float2(-cq, -cq);
      const float2 neg1 = make_float2(-1.f, -1.f);
      const int seg_y = (g.head + y) / V, pos_y = (g.head + y) % V;
      float2 dist2 = make_float2(0.f, 0.f);  // sum over classes of the distance integrand
      typename SegOps<T>::macc lt[PD], ge[PD];
      float za[PD];
#pragma unroll
      for (int j = 0; j < PD; ++j) { lt[j] = SegOps<T>::neg_inf(); ge[j] = SegOps<T>::neg_inf(); za[j] = -INFINITY; }

      const int n_chunks = (g.n_seg + kSegPerChunk - 1) / kSegPerChunk;
      for (int k = 0; k < n_chunks; ++k) {
        float2 z2[kSegPerThread][H], sd2[kSegPerThread][H];
        bool active[kSegPerThread], special[kSegPerThread], edge[kSegPerThread];
        int seg[kSegPerThread];
#pragma unroll
        for (int u = 0; u < kSegPerThread; ++u) {
          seg[u] = k * kSegPerChunk + u * kConsumers + tid;
          active[u] = seg[u] < g.n_seg;
          edge[u] = !(seg[u] >= g.seg_lo && seg[u] < g.seg_hi);
          special[u] = edge[u] || seg[u] == seg_a;
#pragma unroll
          for (int i = 0; i < H; ++i) { z2[u][i] = make_float2(0.f, 0.f); sd2[u][i] = make_float2(0.f, 0.f); }
          if (active[u]) SegOps<T>::unpack2(*reinterpret_cast<const uint4*>(img + (size_t)seg[u] * 16), z2[u]);
        }
        if (stream_peers) {
#pragma unroll
          for (int j = 0; j < P; ++j, ++q) {
            const int st = q % n_stage;
            wait_bounded(&ctrl->ring_full[st], (q / n_stage) & 1, ctrl, a.hdr);
            const char* chunk = ring_base + (size_t)st * kChunkBytes;
#pragma unroll
            for (int u = 0; u < kSegPerThread; ++u) {
              if (!active[u]) continue;
              const uint4 raw = *reinterpret_cast<const uint4*>(chunk + (size_t)(u * kConsumers + tid) * 16);
              float2 d2[H];
              if (!special[u]) {
                float2 v2[H];
                SegOps<T>::unpack2(raw, v2);
#pragma unroll
                for (int i = 0; i < H; ++i) d2[i] = __ffma2_rn(v2[i], neg1, z2[u][i]);
                if (a.want_flags) {
                  const typename SegOps<T>::macc f = SegOps<T>::fold(raw);
                  if (seg[u] < seg_a) lt[j] = SegOps<T>::mmax(lt[j], f); else ge[j] = SegOps<T>::mmax(ge[j], f);
                }
              } else {
                SegPairs<T> zs;
#pragma unroll
                for (int i = 0; i < H; ++i) zs.v[i] = z2[u][i];
                const SlowPeer<T> o = slow_peer<T>(zs, raw, seg[u], g.head, C, a.want_flags ? a_own : -1);
#pragma unroll
                for (int i = 0; i < H; ++i) d2[i] = o.d2[i];
                lt[j] = SegOps<T>::mmax(lt[j], SegOps<T>::from_scalar(o.lt));
                ge[j] = SegOps<T>::mmax(ge[j], SegOps<T>::from_scalar(o.ge));
                za[j] = fmaxf(za[j], o.za);
              }
              if (with_term) {
#pragma unroll
                for (int i = 0; i < H; ++i) {
                  if constexpr (P == 1) sd2[u][i] = d2[i]; else sd2[u][i] = __fadd2_rn(sd2[u][i], d2[i]);
                  if constexpr (PW) dist2 = __ffma2_rn(d2[i], d2[i], dist2);
                }
              }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&ctrl->ring_empty[st]);
          }
        }
        // gradient of this chunk's segments
#pragma unroll
        for (int u = 0; u < kSegPerThread; ++u) {
          if (!active[u]) continue;
          float2 g2[H];
#pragma unroll
          for (int i = 0; i < H; ++i) {
            const float2 e = exp_shift2<T>(z2[u][i], m, l2e2, nml2);
            g2[i] = __ffma2_rn(e, cp2, __ffma2_rn(sd2[u][i], cd2, ncq2));
            if constexpr (!PW) dist2 = __ffma2_rn(sd2[u][i], sd2[u][i], dist2);  // (sum_j d)^2, scaled by 1/P^2 below
          }
          if (seg[u] == seg_y) {
#pragma unroll
            for (int i = 0; i < H; ++i) {
              if (2 * i == pos_y) g2[i].x -= cy;
              if (2 * i + 1 == pos_y) g2[i].y -= cy;
            }
          }
          if (g_img) {
            if (!edge[u]) {
              *reinterpret_cast<uint4*>(g_img + (size_t)seg[u] * 16) = SegOps<T>::pack2(g2);
            } else {
#pragma unroll
              for (int i = 0; i < V; ++i) {
                const int64_t c = (int64_t)seg[u] * V - g.head + i;
                const float gv = (i & 1) ? g2[i >> 1].y : g2[i >> 1].x;
                if (c >= 0 && c < C) reinterpret_cast<T*>(g_img + (size_t)seg[u] * 16)[i] = Elem<T>::from_f32(gv);
              }
            }
          }
        }
      }

      // ---------------- row results
      float dsum[1] = {dist2.x + dist2.y};
      if (with_term) red.sum(dsum);
      uint32_t flags = 0u;
      if (a.want_flags) {
        flags = (a_own == y) ? 1u : 0u;
        if (P >= 1) {
          float mxv[3 * PD];
#pragma unroll
          for (int j = 0; j < PD; ++j) {
            mxv[3 * j] = SegOps<T>::to_float(lt[j]);
            mxv[3 * j + 1] = SegOps<T>::to_float(ge[j]);
            mxv[3 * j + 2] = za[j];
          }
          red.max(mxv);
#pragma unroll
          for (int j = 0; j < PD; ++j)
            if (mxv[3 * j + 2] >= mxv[3 * j + 1] && mxv[3 * j] < mxv[3 * j + 2]) flags |= (2u << j);
        }
      }
      if (tid == 0) {
        float D = 0.f;
        if (with_term) D = PW ? dsum[0] * inv_P / (float)C : dsum[0] * inv_P * inv_P / (float)C;
        a.row_loss[r] = with_term ? fmaf(a.alpha, D, ce) : ce;
        a.row_flags[r] = flags;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&ctrl->own_empty[b]);
    }
  }

  // ---------------- all rows of this CTA are written: scheduler reset and final reduction
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const unsigned int prev = atomicAdd(&a.hdr->sched_done, 1u);
    ctrl->last_flag = (prev == gridDim.x - 1);
    if (ctrl->last_flag) { a.hdr->next_row = 0u; a.hdr->sched_done = 0u; __threadfence(); }  // ready for the next launch
  }
  __syncthreads();
  if (a.fused_finalize && ctrl->last_flag) {
    __threadfence();
    finalize_cta(a, ctrl->fin);
  }
}

// ------------------------------------------------------------------ host side
static bool tma_config(const KArgs& a, int dtype, int smem_optin, TmaCfg* out) {
  const int64_t es = dtype == CODISTILL_F32 ? 4 : 2;
  const int64_t row_bytes = a.classes * es;
  if (a.dist != CODISTILL_DIST_MSE_LOGITS) return false;
  if (!(a.n_peers == 0 || a.n_peers == 1 || a.n_peers == 2 || a.n_peers == 3 || a.n_peers == 7)) return false;
  if (row_bytes < 8192 || a.classes > (int64_t)1 << 24) return false;
  uintptr_t bits = reinterpret_cast<uintptr_t>(a.own) | reinterpret_cast<uintptr_t>(a.grad);
  for (int j = 0; j < a.n_peers; ++j) bits |= reinterpret_cast<uintptr_t>(a.peers[j]);
  if (bits & 15u) return false;
  const int64_t own_buf = ((row_bytes + 32 + 127) / 128) * 128;
  // per-CTA share of the SM's shared memory (1 KiB per CTA is reserved by the system)
  const int64_t avail = (kCtasPerSm == 1 ? (int64_t)smem_optin : ((int64_t)smem_optin + 1024) / kCtasPerSm - 1024) - kCtrlBytes;
  TmaCfg c;
  c.own_buf_bytes = (uint32_t)own_buf;
  const int min_stages = a.n_peers > 0 ? 3 : 1;
  if (2 * own_buf + (int64_t)(a.n_peers > 0 ? 4 : 1) * kChunkBytes <= avail) {
    c.own_bufs = 2;
  } else if (own_buf + (int64_t)min_stages * kChunkBytes <= avail) {
    c.own_bufs = 1;
  } else {
    return false;
  }
  int64_t st = (avail - (int64_t)c.own_bufs * own_buf) / kChunkBytes;
  if (st > kMaxStages) st = kMaxStages;
  c.stages = (int)st;
  c.smem_bytes = (uint32_t)(kCtrlBytes + (int64_t)c.own_bufs * own_buf + (int64_t)c.stages * kChunkBytes);
  *out = c;
  return true;
}

bool tma_supported(const KArgs& a, int dtype, int smem_optin) {
  TmaCfg c;
  return tma_config(a, dtype, smem_optin, &c);
}

template <typename T, int P, bool PW>
static cudaError_t launch_one(const KArgs& a, const TmaCfg& c, int grid, cudaStream_t stream) {
  cudaError_t e = cudaFuncSetAttribute(rows_tma_kernel<T, P, PW>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c.smem_bytes);
  if (e != cudaSuccess) return e;
  rows_tma_kernel<T, P, PW><<<grid, kTmaThreads, c.smem_bytes, stream>>>(a, c);
  return cudaGetLastError();
}

// PW: the loss sums squared pairwise differences (Algorithm 1); otherwise the squared difference to
// the averaged peer.  With one peer the two coincide.
template <typename T>
static cudaError_t launch_dtype(const KArgs& a, const TmaCfg& c, int grid, cudaStream_t stream) {
  const bool pw = a.peer_reduce == CODISTILL_PEERS_PAIRWISE_MEAN;
  switch (a.n_peers) {
    case 0: return launch_one<T, 0, true>(a, c, grid, stream);
    case 1: return launch_one<T, 1, true>(a, c, grid, stream);
    case 2: return pw ? launch_one<T, 2, true>(a, c, grid, stream) : launch_one<T, 2, false>(a, c, grid, stream);
    case 3: return pw ? launch_one<T, 3, true>(a, c, grid, stream) : launch_one<T, 3, false>(a, c, grid, stream);
    case 7: return pw ? launch_one<T, 7, true>(a, c, grid, stream) : launch_one<T, 7, false>(a, c, grid, stream);
    default: return cudaErrorNotSupported;
  }
}

cudaError_t launch_tma(const KArgs& a, int dtype, int num_sms, int smem_optin, cudaStream_t stream) {
  TmaCfg c;
  if (!tma_config(a, dtype, smem_optin, &c)) return cudaErrorNotSupported;
  const int64_t rows = a.row_end - a.row_begin;
  if (rows <= 0) return cudaSuccess;
  const int64_t slots = (int64_t)num_sms * kCtasPerSm;
  const int grid = (int)(rows < slots ? rows : slots);
  return dtype == CODISTILL_F32 ? launch_dtype<float>(a, c, grid, stream) : launch_dtype<__nv_bfloat16>(a, c, grid, stream);
}

}  // namespace codistill
