// Persistent, warp-specialised kernel for long rows ("tma" regime), MSE-on-logits distance.
//
// Each CTA owns one resident row buffer and a ring of stages; as many CTAs as fit run per SM (two
// for 64 KiB rows), so that one CTA's statistics pass overlaps the other's streaming pass.
//   warp 0  scheduler + own-row producer + service: draws row ids from a global counter (mask byte
//           and label are fetched one row ahead), publishes them in a small ring of row-info slots,
//           and moves the own row image into the row buffer piece by piece with 1-D bulk
//           asynchronous copies (cp.async.bulk, no multicast) that complete on one mbarrier per
//           piece.  A piece is refilled for the next row as soon as the consumers are done with it,
//           so the next own row streams in behind the current row's second pass.  The same warp
//           writes the all-zero gradient rows of masked rows and turns the consumers' per-warp
//           partial results of a finished row into the per-row loss and flag word, off the
//           consumers' critical path.
//   warp 1  peer producer: streams the n-1 peer rows chunk by chunk (chunk-major: chunk k of peer
//           0, 1, ..., then chunk k+1) through the ring of stages.
//   others  consumers: one sweep over the resident own row as its pieces land (online softmax:
//           running max, sum exp, sum z, first arg-max), one block reduction, then per chunk:
//           consume the peers from the ring (sum_j (z - z_j), sum_j (z - z_j)^2, what the arg-max
//           agreement needs), write the gradient with 128-bit stores, release the own piece.
// Every logit is read from HBM exactly once and the gradient is written once.
//
// A "row image" is the 16-byte aligned byte range that contains the row: rows whose byte length
// is not a multiple of 16 start at varying offsets `head` inside their first segment.  Segments
// that are only partly inside the row ("edge" segments) take a masked slow path.  Every valid row
// uses the same number of pieces (some possibly empty), so that barrier phases advance uniformly.
#include "bulk_copy.cuh"
#include "common.cuh"
#include "seg_math.cuh"

namespace codistill {

constexpr int kMaxStages = 12;
constexpr int kMaxPieces = 32;
constexpr int kInfoSlots = 4;
constexpr int kCtrlBytes = 8192;        // control block, then kZeroBytes of zeros
constexpr int kZeroBytes = 2048;        // source of the bulk stores that write all-zero gradient rows
constexpr int kProducerThreads = 64;   // warp 0: scheduler + own row, warp 1: peers + service
constexpr int kSegPerThread = 2;       // 16-byte segments per consumer thread per chunk
constexpr int kMaxConsumerWarps = 16;
constexpr uint32_t kBulkPieceBytes = 32768;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;  // bounded waits: 2 s, then CODISTILL_DEV_TIMEOUT
constexpr unsigned long long kDrainLimitNs = 50000000ull;   // per barrier when a producer leaves: 50 ms

struct TmaCfg {
  int consumer_warps;  // 8 (two CTAs per SM) or 16 (one CTA per SM)
  int ctas_per_sm;
  int stages;          // ring stages of chunk_bytes each
  int pieces;          // chunks per row image (same for every row of the call)
  uint32_t chunk_bytes;
  uint32_t own_buf_bytes;
  uint32_t smem_bytes;
};

struct RowInfo {
  long long row;  // global row id, -1 = no more rows
  int valid;
  int label;
};

struct Ctrl {  // lives at the start of dynamic shared memory
  uint64_t own_full[kMaxPieces];
  uint64_t own_empty[kMaxPieces];
  uint64_t ring_full[kMaxStages];
  uint64_t ring_empty[kMaxStages];
  uint64_t info_full[kInfoSlots];
  uint64_t info_empty[kInfoSlots];
  RowInfo info[kInfoSlots];
  int abort_flag;
  int last_flag;
  uint64_t end_full[2];    // consumers -> service warp: partial results of a row are in endred[par]
  uint64_t end_empty[2];   // service warp -> consumers: endred[par] may be overwritten
  alignas(16) float red[2][kMaxConsumerWarps * 4];  // reduction scratch of the consumers, two alternating halves
  float endred[2][kMaxConsumerWarps * 24];  // per-warp partials of the end-of-row reduction
  float end_ce[2];                          // task loss of the row
  int end_correct[2];                       // arg-max == label
  double fin[32];
};
static_assert(sizeof(Ctrl) <= kCtrlBytes - kZeroBytes, "control block fits its slot");

// Wait for a phase of an mbarrier, but never for ever: after kWaitLimitNs the CTA-wide abort flag
// and the device status are set and every later wait returns early (results are then invalid).  The
// producer warps wait most of the time and have slack (ring stages, row pieces ahead): they back off
// between polls, so that their polling does not take issue slots from the consumers.
__device__ __forceinline__ void wait_bounded(uint64_t* bar, uint32_t parity, Ctrl* ctrl, WsHeader* hdr) {
  if (mbar_try_wait(bar, parity)) return;
  mbar_wait_limited(bar, parity, &ctrl->abort_flag, &hdr->status, CODISTILL_DEV_TIMEOUT, kWaitLimitNs, true,
                    threadIdx.x < kProducerThreads);
}
// Last wait of a producer warp on a barrier it armed: also after an abort the copies that complete on it
// get one further, shorter interval to land, so that the CTA does not end with a copy into its shared
// memory still in flight.
__device__ __forceinline__ void wait_drain(uint64_t* bar, uint32_t parity, Ctrl* ctrl, WsHeader* hdr) {
  if (mbar_try_wait(bar, parity)) return;
  mbar_wait_limited(bar, parity, &ctrl->abort_flag, &hdr->status, CODISTILL_DEV_TIMEOUT, kDrainLimitNs, false, true);
}

// Block reductions among the NCW * 32 consumer threads (one named barrier each).
template <int NCW>
struct ConsumerReduce {
  Ctrl* ctrl;
  int toggle;
  int warp, lane;  // consumer warp index 0..NCW-1
  __device__ __forceinline__ static void bar() { asm volatile("bar.sync 1, %0;" ::"n"(NCW * 32) : "memory"); }
  template <int N>
  __device__ __forceinline__ void sum(float (&v)[N]) {
    float* s = ctrl->red[toggle];
#pragma unroll
    for (int k = 0; k < N; ++k) {
      v[k] = warp_sum(v[k]);
      if (lane == 0) s[k * NCW + warp] = v[k];
    }
    bar();
#pragma unroll
    for (int k = 0; k < N; ++k) v[k] = warp_sum(lane < NCW ? s[k * NCW + lane] : 0.f);
    toggle ^= 1;
  }
  template <int N>
  __device__ __forceinline__ void max(float (&v)[N]) {
    float* s = ctrl->red[toggle];
#pragma unroll
    for (int k = 0; k < N; ++k) {
      v[k] = warp_max(v[k]);
      if (lane == 0) s[k * NCW + warp] = v[k];
    }
    bar();
#pragma unroll
    for (int k = 0; k < N; ++k) v[k] = warp_max(lane < NCW ? s[k * NCW + lane] : -INFINITY);
    toggle ^= 1;
  }
  // larger value wins; on equal values the smaller index wins
  __device__ __forceinline__ void argmax(float& v, int& i) {
    float* s = ctrl->red[toggle];
    warp_argmax(v, i);
    if (lane == 0) { s[warp] = v; reinterpret_cast<int*>(s)[NCW + warp] = i; }
    bar();
    v = lane < NCW ? s[lane] : -INFINITY;
    i = lane < NCW ? reinterpret_cast<int*>(s)[NCW + lane] : 0x7fffffff;
    warp_argmax(v, i);
    toggle ^= 1;
  }
  __device__ __forceinline__ int min_int(int v) {
    int* s = reinterpret_cast<int*>(ctrl->red[toggle]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = ::min(v, __shfl_xor_sync(0xffffffffu, v, o));
    if (lane == 0) s[warp] = v;
    bar();
    v = lane < NCW ? s[lane] : 0x7fffffff;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = ::min(v, __shfl_xor_sync(0xffffffffu, v, o));
    toggle ^= 1;
    return v;
  }
};

// ------------------------------------------------------------------ producer helpers
// Moves bytes [begin, end) of a row image whose start is `src` (16-byte aligned) to `dst` (the
// shared-memory address of byte `begin`), completing on `bar` (one arrival + the byte count).
// `tma_limit` is where whole-segment reads must stop: the elements between tma_limit and valid_end
// (a partial last segment at the very end of a tensor) are fetched with plain loads by the lanes of
// the producer warp.  Called by a whole producer warp.
template <typename T>
__device__ __forceinline__ void produce_copy(char* dst, const char* src, uint32_t begin, uint32_t end, uint32_t tma_limit,
                                             uint32_t valid_end, uint64_t* bar, int lane) {
  const uint32_t tma_end = end < tma_limit ? end : tma_limit;
  if (end > tma_limit) {  // partial last segment that must not be read as a whole
    const uint32_t first = tma_limit > begin ? tma_limit : begin;
    const uint32_t off = first + (uint32_t)lane * (uint32_t)sizeof(T);
    if (off < valid_end && off < end) *reinterpret_cast<T*>(dst + (off - begin)) = *reinterpret_cast<const T*>(src + off);
    __syncwarp();
  }
  if (lane == 0) {
    const uint32_t bytes = tma_end > begin ? tma_end - begin : 0u;
    mbar_arrive_expect_tx(bar, bytes);
    for (uint32_t o = 0; o < bytes; o += kBulkPieceBytes) {
      const uint32_t piece = bytes - o < kBulkPieceBytes ? bytes - o : kBulkPieceBytes;
      bulk_g2s(dst + o, src + begin + o, piece, bar);
    }
  }
}

// Per-row quantities both producers derive from the row id.
struct RowCopy {
  uint32_t img_bytes, valid_end, tma_limit;
  int64_t row_off;  // image start relative to the tensor, in bytes
};
template <typename T>
__device__ __forceinline__ RowCopy row_copy(const KArgs& a, long long r) {
  constexpr int ES = (int)sizeof(T);
  const int64_t lr = r - a.row_begin;
  const RowGeom g = row_geom<T>(lr, a.row_stride, a.classes);
  RowCopy c;
  c.img_bytes = (uint32_t)g.n_seg * 16u;
  c.valid_end = (uint32_t)(g.head + a.classes) * ES;
  // The last row of the whole call may end inside a segment that reaches past the tensor.
  const bool clip = (r == a.rows_total - 1) && ((a.row_stride - a.classes) * ES < 16) && (c.valid_end & 15u);
  c.tma_limit = clip ? (c.valid_end & ~15u) : c.img_bytes;
  c.row_off = lr * a.row_stride * ES - (int64_t)g.head * ES;
  return c;
}

// First column of segment `s` whose value equals m, or INT_MAX.
template <typename T>
__device__ __noinline__ int first_equal(const char* img, int s, int head, int64_t C, float m) {
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
// T: element type; P: number of peers (compile time); PW: the loss sums squared pairwise differences
// (otherwise the squared difference to the averaged peer); NCW: consumer warps per CTA.
template <typename T, int P, bool PW, int NCW>
__global__ void __launch_bounds__(NCW * 32 + kProducerThreads, NCW == 8 ? 2 : 1)
rows_tma_kernel(const __grid_constant__ KArgs a, const TmaCfg cfg) {
  constexpr int V = SegOps<T>::V;
  constexpr int H = SegOps<T>::H;
  constexpr int PD = P > 0 ? P : 1;
  constexpr int ES = (int)sizeof(T);
  constexpr int kConsumers = NCW * 32;
  constexpr int kSegPerChunk = kConsumers * kSegPerThread;
  constexpr uint32_t kChunkBytes = kSegPerChunk * 16;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  Ctrl* ctrl = reinterpret_cast<Ctrl*>(smem_raw);
  char* own_buf = reinterpret_cast<char*>(smem_raw) + kCtrlBytes;
  char* ring_base = own_buf + cfg.own_buf_bytes;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_stage = cfg.stages, n_pieces = cfg.pieces;
  const int64_t C = a.classes;
  const bool with_term = (P >= 1 && a.alpha != 0.f);
  const bool stream_peers = (P >= 1) && (with_term || a.want_flags);

  if (threadIdx.x == 0) {
    for (int k = 0; k < kMaxPieces; ++k) { mbar_init(&ctrl->own_full[k], 1); mbar_init(&ctrl->own_empty[k], NCW); }
    for (int s = 0; s < kMaxStages; ++s) { mbar_init(&ctrl->ring_full[s], 1); mbar_init(&ctrl->ring_empty[s], NCW); }
    for (int s = 0; s < kInfoSlots; ++s) { mbar_init(&ctrl->info_full[s], 1); mbar_init(&ctrl->info_empty[s], NCW + 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(&ctrl->end_full[s], NCW); mbar_init(&ctrl->end_empty[s], 1); }
    ctrl->abort_flag = 0;
    ctrl->last_flag = 0;
    mbar_init_fence();
  }
  char* zero_region = reinterpret_cast<char*>(smem_raw) + (kCtrlBytes - kZeroBytes);
  for (int i = threadIdx.x * 16; i < kZeroBytes; i += blockDim.x * 16) *reinterpret_cast<uint4*>(zero_region + i) = make_uint4(0u, 0u, 0u, 0u);
  fence_proxy_async_shared();  // the zeros are read by bulk copies later
  wait_for_prior_grid();  // from here on the workspace header and the valid-row counts are read
  __syncthreads();

  if (warp == 0) {
    // ============================== scheduler + own-row producer ==============================
    // Row ids come from a global counter.  The counter and the row's mask byte and label are fetched
    // two and one iterations ahead (lane 0), so that their latency never sits between two rows.
    long long t_next = 0, t_next2 = 0;
    int mask_next = 0, label_next = 0;
    if (lane == 0) {
      t_next = a.row_begin + (long long)atomicAdd(&a.hdr->next_row, 1u);
      t_next2 = a.row_begin + (long long)atomicAdd(&a.hdr->next_row, 1u);
      if (t_next < a.row_end) { mask_next = a.mask ? a.mask[t_next] : 1; label_next = a.labels[t_next]; }
    }
    const float inv_P = P >= 1 ? 1.f / (float)P : 0.f;
    // Turns the consumers' per-warp partials of valid row number `vv` into its loss and flag word.
    auto finish_row = [&](int vv, long long row) {
      const int par = vv & 1;
      wait_bounded(&ctrl->end_full[par], (uint32_t)(vv >> 1) & 1u, ctrl, a.hdr);
      const float* er = ctrl->endred[par];
      const float dsum = warp_sum(lane < NCW ? er[lane] : 0.f);
      uint32_t flags = 0u;
      if (a.want_flags) {
        flags = ctrl->end_correct[par] ? 1u : 0u;
#pragma unroll
        for (int j = 0; j < P; ++j) {
          const float ltv = warp_max(lane < NCW ? er[(1 + 3 * j) * NCW + lane] : -INFINITY);
          const float gev = warp_max(lane < NCW ? er[(2 + 3 * j) * NCW + lane] : -INFINITY);
          const float zav = warp_max(lane < NCW ? er[(3 + 3 * j) * NCW + lane] : -INFINITY);
          if (zav >= gev && ltv < zav) flags |= (2u << j);
        }
      }
      const float ce = ctrl->end_ce[par];
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(&ctrl->end_empty[par]);
        float D = 0.f;
        if (with_term) D = PW ? dsum * inv_P / (float)C : dsum * inv_P * inv_P / (float)C;
        a.row_loss[row] = with_term ? fmaf(a.alpha, D, ce) : ce;
        a.row_flags[row] = flags;
      }
    };
    int v = 0;  // valid rows copied so far
    long long prev_row[2] = {-1, -1};  // rows whose results are still to be finished (valid rows v-2, v-1)
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
      const bool more = r < a.row_end;
      const bool valid = more && mask_v != 0 && label_v >= 0 && (int64_t)label_v < C;
      const int slot = it % kInfoSlots;
      if (it >= kInfoSlots) wait_bounded(&ctrl->info_empty[slot], ((it / kInfoSlots) - 1) & 1, ctrl, a.hdr);
      if (lane == 0) {
        ctrl->info[slot].row = more ? r : -1;
        ctrl->info[slot].valid = valid;
        ctrl->info[slot].label = label_v;
        mbar_arrive(&ctrl->info_full[slot]);
      }
      if (!more) break;
      if (!valid) {  // masked row: zero gradient, no loss, no counts; nothing is copied for it
        if (a.grad) {
          // whole segments inside the row: bulk copies of zeros; the ragged first / last segments: element stores
          const int64_t lr = r - a.row_begin;
          const RowGeom g = row_geom<T>(lr, a.row_stride, C);
          char* g_img = reinterpret_cast<char*>(a.grad) + lr * a.row_stride * ES - (int64_t)g.head * ES;
          if (lane == 0) {
            const uint32_t lo = (uint32_t)g.seg_lo * 16u, hi = (uint32_t)g.seg_hi * 16u;
            for (uint32_t o = lo; o < hi; o += kZeroBytes) bulk_s2g(g_img + o, zero_region, hi - o < (uint32_t)kZeroBytes ? hi - o : (uint32_t)kZeroBytes);
            bulk_commit_group();
          }
          if (lane < 2) {
            const int s = lane == 0 ? 0 : g.n_seg - 1;
            if ((lane == 0 && g.seg_lo > 0) || (lane == 1 && g.seg_hi < g.n_seg && (g.n_seg > 1 || g.seg_lo == 0))) {
#pragma unroll
              for (int i = 0; i < V; ++i) {
                const int64_t c = (int64_t)s * V - g.head + i;
                if (c >= 0 && c < C) reinterpret_cast<T*>(g_img + (size_t)s * 16)[i] = Elem<T>::from_f32(0.f);
              }
            }
          }
        }
        if (lane == 0) { a.row_loss[r] = 0.f; a.row_flags[r] = 0u; }
        continue;
      }
      // The consumers are at most one row behind this warp, so valid row v-2 is complete: finish it
      // before feeding row v (the consumers reuse its partial-result slot at the end of row v).
      if (v >= 2) finish_row(v - 2, prev_row[v & 1]);
      prev_row[v & 1] = r;
      const RowCopy rc = row_copy<T>(a, r);
      const char* src = reinterpret_cast<const char*>(a.own) + rc.row_off;
      for (int k = 0; k < n_pieces; ++k) {
        if (v >= 1) wait_bounded(&ctrl->own_empty[k], (v - 1) & 1, ctrl, a.hdr);
        const uint32_t begin = (uint32_t)k * kChunkBytes;
        uint32_t end = begin + kChunkBytes < rc.img_bytes ? begin + kChunkBytes : rc.img_bytes;
        if (end < begin) end = begin;  // empty piece of a shorter row image
        produce_copy<T>(own_buf + begin, src, begin, end, rc.tma_limit, rc.valid_end, &ctrl->own_full[k], lane);
      }
      ++v;
    }
    // results of the last two valid rows
    if (v >= 2) finish_row(v - 2, prev_row[v & 1]);
    if (v >= 1) finish_row(v - 1, prev_row[(v - 1) & 1]);
    if (lane == 0) bulk_wait_all_groups();  // zero rows are written
    // Before leaving, make sure no copy armed by this warp is still in flight (bounded).
    if (v >= 1)
      for (int k = 0; k < n_pieces; ++k) wait_drain(&ctrl->own_full[k], (v - 1) & 1, ctrl, a.hdr);
  } else if (warp == 1) {
    // ============================== peer producer ==============================
    uint32_t q = 0;          // ring items issued so far
    int st = 0;              // stage of the next item
    uint32_t st_phase = 0;   // phase bit of that stage's next use
    for (int it = 0;; ++it) {
      const int slot = it % kInfoSlots;
      wait_bounded(&ctrl->info_full[slot], (it / kInfoSlots) & 1, ctrl, a.hdr);
      const long long r = ctrl->info[slot].row;
      const bool valid = ctrl->info[slot].valid != 0;
      __syncwarp();
      if (lane == 0) mbar_arrive(&ctrl->info_empty[slot]);
      if (r < 0) break;
      if (!valid || !stream_peers) continue;
      const RowCopy rc = row_copy<T>(a, r);
      for (int k = 0; k < n_pieces; ++k) {
        const uint32_t begin = (uint32_t)k * kChunkBytes;
        uint32_t end = begin + kChunkBytes < rc.img_bytes ? begin + kChunkBytes : rc.img_bytes;
        if (end < begin) end = begin;
#pragma unroll 1
        for (int j = 0; j < P; ++j, ++q) {
          if (q >= (uint32_t)n_stage) wait_bounded(&ctrl->ring_empty[st], st_phase ^ 1u, ctrl, a.hdr);
          produce_copy<T>(ring_base + (size_t)st * kChunkBytes, reinterpret_cast<const char*>(a.peers[j]) + rc.row_off, begin, end,
                          rc.tma_limit, rc.valid_end, &ctrl->ring_full[st], lane);
          if (++st == n_stage) { st = 0; st_phase ^= 1u; }
        }
      }
    }
    for (uint32_t i = 0; i < (uint32_t)n_stage && i < q; ++i) {
      const uint32_t qi = q - 1 - i;
      wait_drain(&ctrl->ring_full[qi % n_stage], (qi / n_stage) & 1, ctrl, a.hdr);
    }
  } else {
    // ============================== consumer warps ==============================
    const int tid = threadIdx.x - kProducerThreads;
    ConsumerReduce<NCW> red{ctrl, 0, warp - 2, lane};
    float w = 1.f;
    if (a.reduction == CODISTILL_REDUCE_MEAN_VALID) {
      const int64_t nv = total_valid(a);
      w = 1.f / (float)(nv > 1 ? nv : 1);
    }
    const float inv_P = P >= 1 ? 1.f / (float)P : 0.f;
    const float inv_C = 1.f / (float)C;
    int st = 0;              // ring stage of the next item
    uint32_t st_phase = 0;   // its phase bit
    int v = 0;               // valid rows processed so far
    for (int it = 0;; ++it) {
      const int slot = it % kInfoSlots;
      wait_bounded(&ctrl->info_full[slot], (it / kInfoSlots) & 1, ctrl, a.hdr);
      const long long r = ctrl->info[slot].row;
      const bool valid = ctrl->info[slot].valid != 0;
      const int y = ctrl->info[slot].label;
      __syncwarp();
      if (lane == 0) mbar_arrive(&ctrl->info_empty[slot]);
      if (r < 0) break;
      const int64_t lr = r - a.row_begin;
      const RowGeom g = row_geom<T>(lr, a.row_stride, C);
      const char* img = own_buf;
      char* g_img = a.grad ? reinterpret_cast<char*>(a.grad) + lr * a.row_stride * ES - (int64_t)g.head * ES : nullptr;

      if (!valid) continue;  // masked rows are written by the service warp
      // Bit k set: in piece k this thread has a segment that needs care (ragged edge of the row, or
      // past its end); all other pieces take straight-line code.
      uint32_t odd_sweep = 0u;
      {
        auto mark = [&](int s) {
          if (((s % kSegPerChunk) % kConsumers) == tid) odd_sweep |= 1u << (s / kSegPerChunk);
        };
        if (g.seg_lo > 0) mark(0);
        if (g.seg_hi < g.n_seg) mark(g.n_seg - 1);
        const int room = g.n_seg - (kSegPerThread - 1) * kConsumers - tid;  // segments before this thread's last lane runs out
        const int k_bad = room > 0 ? (room + kSegPerChunk - 1) / kSegPerChunk : 0;
        if (k_bad < 32) odd_sweep |= ~0u << k_bad;
      }
      const uint32_t own_parity = (uint32_t)v & 1u;

      // ---------------- one sweep over the own row, piece by piece as it lands (online softmax):
      // running maximum `best` with the first segment that attains it (a thread visits its segments
      // in rising order, so a strict comparison keeps the first), sum exp(z - best), sum z.
      const float2 l2e2 = make_float2(kLog2e, kLog2e);
      float best = -3.0e38f;  // finite, so that the first rescale is exp2(-huge) = 0 and never NaN
      int best_seg = 0x7fffffff;
      float2 s2[H], zs2[H];
#pragma unroll
      for (int i = 0; i < H; ++i) { s2[i] = make_float2(0.f, 0.f); zs2[i] = make_float2(0.f, 0.f); }
      float s_edge = 0.f, z_edge = 0.f;  // contributions of ragged edge segments (relative to `best`)
      for (int k = 0; k < n_pieces; ++k) {
        wait_bounded(&ctrl->own_full[k], own_parity, ctrl, a.hdr);
        if (!((odd_sweep >> k) & 1u)) {
          // ---- straight-line path: all of this thread's segments of the piece lie inside the row
          const uint32_t off = (uint32_t)k * kChunkBytes + (uint32_t)tid * 16u;
          uint4 rw[kSegPerThread];
          const float old_best = best;
#pragma unroll
          for (int u = 0; u < kSegPerThread; ++u) {
            rw[u] = *reinterpret_cast<const uint4*>(img + off + u * (kConsumers * 16));
            const float fm = SegOps<T>::to_float(SegOps<T>::fold(rw[u]));
            if (fm > best) { best = fm; best_seg = k * kSegPerChunk + u * kConsumers + tid; }
          }
          const float sc = rescale_exp2<T>((old_best - best) * kLog2e);
          const float2 sc2 = make_float2(sc, sc);
          const float2 nmk = make_float2(-best * kLog2e, -best * kLog2e);
          s_edge *= sc;
#pragma unroll
          for (int i = 0; i < H; ++i) s2[i] = __fmul2_rn(s2[i], sc2);
#pragma unroll
          for (int u = 0; u < kSegPerThread; ++u) {
            float2 z2[H];
            SegOps<T>::unpack2(rw[u], z2);
#pragma unroll
            for (int i = 0; i < H; ++i) {
              s2[i] = __fadd2_rn(s2[i], exp_shift2<T>(z2[i], best, l2e2, nmk));
              zs2[i] = __fadd2_rn(zs2[i], z2[i]);
            }
          }
          continue;
        }
        uint4 raw[kSegPerThread];
        bool inner[kSegPerThread], ragged[kSegPerThread];
        const float old = best;
#pragma unroll
        for (int u = 0; u < kSegPerThread; ++u) {
          const int s = k * kSegPerChunk + u * kConsumers + tid;
          inner[u] = s >= g.seg_lo && s < g.seg_hi;
          ragged[u] = !inner[u] && s < g.n_seg;
          float fm = -3.0e38f;
          if (inner[u] || ragged[u]) raw[u] = *reinterpret_cast<const uint4*>(img + (size_t)s * 16);
          if (inner[u]) {
            fm = SegOps<T>::to_float(SegOps<T>::fold(raw[u]));
          } else if (ragged[u]) {
            float z[V];
            SegOps<T>::unpack(raw[u], z);
#pragma unroll
            for (int i = 0; i < V; ++i) {
              const int64_t c = (int64_t)s * V - g.head + i;
              if (c >= 0 && c < C) fm = fmaxf(fm, z[i]);
            }
          }
          if (fm > best) { best = fm; best_seg = s; }
        }
        // rescale what was summed so far to the new reference (factor 1 when it did not move)
        const float scale = rescale_exp2<T>((old - best) * kLog2e);
        const float2 scale2 = make_float2(scale, scale);
        const float2 nml2k = make_float2(-best * kLog2e, -best * kLog2e);
        s_edge *= scale;
#pragma unroll
        for (int i = 0; i < H; ++i) s2[i] = __fmul2_rn(s2[i], scale2);
#pragma unroll
        for (int u = 0; u < kSegPerThread; ++u) {
          const int s = k * kSegPerChunk + u * kConsumers + tid;
          if (inner[u]) {
            float2 z2[H];
            SegOps<T>::unpack2(raw[u], z2);
#pragma unroll
            for (int i = 0; i < H; ++i) {
              s2[i] = __fadd2_rn(s2[i], exp_shift2<T>(z2[i], best, l2e2, nml2k));
              zs2[i] = __fadd2_rn(zs2[i], z2[i]);
            }
          } else if (ragged[u]) {
            float z[V];
            SegOps<T>::unpack(raw[u], z);
#pragma unroll
            for (int i = 0; i < V; ++i) {
              const int64_t c = (int64_t)s * V - g.head + i;
              if (c >= 0 && c < C) {
                s_edge += exp_shift2<T>(make_float2(z[i], z[i]), best, l2e2, nml2k).x;
                z_edge += z[i];
              }
            }
          }
        }
      }
      float s_t = s_edge, z_t = z_edge;
#pragma unroll
      for (int i = 0; i < H; ++i) { s_t += s2[i].x + s2[i].y; z_t += zs2[i].x + zs2[i].y; }
      // block reduction in one round: maximum with its first segment, then the sums rescaled to it
      float m = best;
      int m_seg = best_seg;
      float S, sum_z;
      {
        // within the warp: the maximum by an integer reduction on an order-preserving image of the
        // float (-0 is folded onto +0 first: they tie), its first segment by a second one; the sums
        // by shuffles
        const unsigned key = float_order_key(best + 0.f);
        const unsigned key_w = __reduce_max_sync(0xffffffffu, key);
        const int seg_w = (int)__reduce_min_sync(0xffffffffu, key == key_w ? (unsigned)best_seg : 0x7fffffffu);
        const float m_w = float_from_order_key(key_w);
        const float sw = warp_sum(s_t * rescale_exp2<T>((best - m_w) * kLog2e));
        const float zw = warp_sum(z_t);
        float4* sc = reinterpret_cast<float4*>(ctrl->red[red.toggle]);
        if (lane == 0) sc[red.warp] = make_float4(m_w, __int_as_float(seg_w), sw, zw);
        ConsumerReduce<NCW>::bar();
        // across warps: every thread combines the NCW partials itself (broadcast reads, fixed order)
        float4 part[NCW];
#pragma unroll
        for (int wv = 0; wv < NCW; ++wv) part[wv] = sc[wv];
        m = part[0].x;
        m_seg = __float_as_int(part[0].y);
#pragma unroll
        for (int wv = 1; wv < NCW; ++wv) argmax_combine(m, m_seg, part[wv].x, __float_as_int(part[wv].y));
        S = 0.f;
        sum_z = 0.f;
#pragma unroll
        for (int wv = 0; wv < NCW; ++wv) {
          S += part[wv].z * rescale_exp2<T>((part[wv].x - m) * kLog2e);
          sum_z += part[wv].w;
        }
        red.toggle ^= 1;
      }
      if (m_seg >= g.n_seg) m_seg = 0;  // NaN rows: keep the read below inside the row image
      const float2 nml2 = make_float2(-m * kLog2e, -m * kLog2e);
      // every thread reads the winning segment: first column that attains the maximum
      const int a_own = first_equal<T>(img, m_seg, g.head, C, m);
      const int seg_a = a.want_flags ? m_seg : -1;
      const float zy = Elem<T>::to_f32(reinterpret_cast<const T*>(img)[g.head + y]);
      float ce = 0.f;  // task loss of the row: only the thread that publishes it computes it
      if (red.warp == 0 && lane == 0) ce = (m + logf(S)) - (1.f - a.eps) * zy - (a.eps * inv_C) * sum_z;

      // ---------------- stream the peers chunk by chunk, write the gradient, release the own pieces
      const float cp = w * __frcp_rn(S);                                          // e_c -> w * p_c
      const float cd = with_term ? w * a.alpha * (2.f * inv_C) * inv_P : 0.f;     // sum_j d -> w * alpha * dD
      const float cq = w * a.eps * inv_C;
      const float cy = w * (1.f - a.eps);
      const float2 cp2 = make_float2(cp, cp), cd2 = make_float2(cd, cd), ncq2 = make_float2(-cq, -cq);
      const float2 neg1 = make_float2(-1.f, -1.f);
      const int seg_y = (g.head + y) / V, pos_y = (g.head + y) % V;
      float2 dist2 = make_float2(0.f, 0.f);  // sum over classes of the distance integrand
      typename SegOps<T>::macc lt[PD], ge[PD];
      float za[PD];
#pragma unroll
      for (int j = 0; j < PD; ++j) { lt[j] = SegOps<T>::neg_inf(); ge[j] = SegOps<T>::neg_inf(); za[j] = -INFINITY; }

      // The thread that holds the label column or the own arg-max column patches its straight-line
      // code for that one segment (bit k of spec_y / spec_a: it is in piece k); only ragged pieces
      // take the general code.
      const uint32_t odd = odd_sweep;
      const uint32_t spec_y = (((seg_y % kSegPerChunk) % kConsumers) == tid) ? 1u << (seg_y / kSegPerChunk) : 0u;
      const uint32_t spec_a = (seg_a >= 0 && ((seg_a % kSegPerChunk) % kConsumers) == tid) ? 1u << (seg_a / kSegPerChunk) : 0u;
      const int u_y = (seg_y % kSegPerChunk) / kConsumers, u_a = seg_a >= 0 ? (seg_a % kSegPerChunk) / kConsumers : 0;
      const bool lean_ok = with_term && g_img != nullptr;   // without counters seg_a is -1: the agreement maxima are kept but never read
      float2 dist2b = make_float2(0.f, 0.f);
      const uint32_t tid16 = (uint32_t)tid * 16u;

      for (int k = 0; k < n_pieces; ++k) {
        if (lean_ok && !((odd >> k) & 1u)) {
          // ---- straight-line path: every segment of this thread lies inside the row, away from the
          // arg-max and label columns
          const uint32_t off = (uint32_t)k * kChunkBytes + tid16;
          float2 z2[kSegPerThread][H], sd2[kSegPerThread][H];
          bool before[kSegPerThread];
#pragma unroll
          for (int u = 0; u < kSegPerThread; ++u) {
            SegOps<T>::unpack2(*reinterpret_cast<const uint4*>(img + off + u * (kConsumers * 16)), z2[u]);
            before[u] = (k * kSegPerChunk + u * kConsumers + tid) < seg_a;
          }
#pragma unroll
          for (int j = 0; j < P; ++j) {
            wait_bounded(&ctrl->ring_full[st], st_phase, ctrl, a.hdr);
            const char* chunk = ring_base + (uint32_t)st * kChunkBytes + tid16;
            uint4 raw[kSegPerThread];
#pragma unroll
            for (int u = 0; u < kSegPerThread; ++u) raw[u] = *reinterpret_cast<const uint4*>(chunk + u * (kConsumers * 16));
#pragma unroll
            for (int u = 0; u < kSegPerThread; ++u) {
              float2 v2[H];
              SegOps<T>::unpack2(raw[u], v2);
#pragma unroll
              for (int i = 0; i < H; ++i) {
                const float2 d = __ffma2_rn(v2[i], neg1, z2[u][i]);
                if (P == 1 || j == 0) sd2[u][i] = d; else sd2[u][i] = __fadd2_rn(sd2[u][i], d);
                if constexpr (PW) { if (i & 1) dist2b = __ffma2_rn(d, d, dist2b); else dist2 = __ffma2_rn(d, d, dist2); }
              }
              const typename SegOps<T>::macc f = SegOps<T>::fold(raw[u]);
              lt[j] = before[u] ? SegOps<T>::mmax(lt[j], f) : lt[j];
              ge[j] = before[u] ? ge[j] : SegOps<T>::mmax(ge[j], f);
            }
            if ((spec_a >> k) & 1u) {
              // The segment of the own arg-max column a went to ge[] as a whole.  The peer's value at a and
              // the largest value before a inside the segment settle the rest: with them in za[] and lt[],
              // "za >= ge and lt < za" holds exactly when the peer's first arg-max is a.
              float vv[V];
              SegOps<T>::unpack(u_a == 0 ? raw[0] : raw[kSegPerThread - 1], vv);
              float pre = -INFINITY;
#pragma unroll
              for (int i = 0; i < V; ++i) {
                const int c = seg_a * V - g.head + i;
                if (c < a_own) pre = fmaxf(pre, vv[i]);
                if (c == a_own) za[j] = vv[i];
              }
              lt[j] = SegOps<T>::mmax(lt[j], SegOps<T>::from_scalar(pre));
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&ctrl->ring_empty[st]);
            if (++st == n_stage) { st = 0; st_phase ^= 1u; }
          }
#pragma unroll
          for (int u = 0; u < kSegPerThread; ++u) {
            float2 g2[H];
#pragma unroll
            for (int i = 0; i < H; ++i) {
              const float2 e = exp_shift2<T>(z2[u][i], m, l2e2, nml2);
              g2[i] = __ffma2_rn(e, cp2, __ffma2_rn(sd2[u][i], cd2, ncq2));
              if constexpr (!PW) dist2 = __ffma2_rn(sd2[u][i], sd2[u][i], dist2);
            }
            if (((spec_y >> k) & 1u) && u == u_y) {  // the label column: q_y carries the extra 1 - eps
#pragma unroll
              for (int i = 0; i < H; ++i) {
                if (2 * i == pos_y) g2[i].x -= cy;
                if (2 * i + 1 == pos_y) g2[i].y -= cy;
              }
            }
            *reinterpret_cast<uint4*>(g_img + off + u * (kConsumers * 16)) = SegOps<T>::pack2(g2);
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(&ctrl->own_empty[k]);
          continue;
        }
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
        bool all_fast = with_term;
#pragma unroll
        for (int u = 0; u < kSegPerThread; ++u) all_fast = all_fast && active[u] && !special[u];
        if (stream_peers) {
#pragma unroll
          for (int j = 0; j < P; ++j) {
            wait_bounded(&ctrl->ring_full[st], st_phase, ctrl, a.hdr);
            const char* chunk = ring_base + (size_t)st * kChunkBytes;
            if (all_fast) {  // both segments lie wholly inside the row and away from the arg-max column
              uint4 raw[kSegPerThread];
#pragma unroll
              for (int u = 0; u < kSegPerThread; ++u)
                raw[u] = *reinterpret_cast<const uint4*>(chunk + (size_t)(u * kConsumers + tid) * 16);
#pragma unroll
              for (int u = 0; u < kSegPerThread; ++u) {
                float2 v2[H];
                SegOps<T>::unpack2(raw[u], v2);
#pragma unroll
                for (int i = 0; i < H; ++i) {
                  const float2 d = __ffma2_rn(v2[i], neg1, z2[u][i]);
                  if constexpr (P == 1) sd2[u][i] = d; else sd2[u][i] = __fadd2_rn(sd2[u][i], d);
                  if constexpr (PW) dist2 = __ffma2_rn(d, d, dist2);
                }
                if (a.want_flags) {
                  const typename SegOps<T>::macc f = SegOps<T>::fold(raw[u]);
                  const bool before = seg[u] < seg_a;
                  lt[j] = before ? SegOps<T>::mmax(lt[j], f) : lt[j];
                  ge[j] = before ? ge[j] : SegOps<T>::mmax(ge[j], f);
                }
              }
            } else
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
            if (++st == n_stage) { st = 0; st_phase ^= 1u; }
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
        // this piece of the own row is no longer needed: the producer may refill it
        __syncwarp();
        if (lane == 0) mbar_arrive(&ctrl->own_empty[k]);
      }
      ++v;

      // ---------------- row results: per-warp partials go to the service warp, nobody waits here
      {
        const int par = (v - 1) & 1;  // v was advanced above
        const int done = v - 1;       // index of this valid row
        float part[1 + 3 * PD];
        part[0] = warp_sum((dist2.x + dist2.y) + (dist2b.x + dist2b.y));
#pragma unroll
        for (int j = 0; j < PD; ++j) {
          part[1 + 3 * j] = warp_max_redux(SegOps<T>::to_float(lt[j]));
          part[2 + 3 * j] = warp_max_redux(SegOps<T>::to_float(ge[j]));
          part[3 + 3 * j] = warp_max_redux(za[j]);
        }
        if (done >= 2) wait_bounded(&ctrl->end_empty[par], (uint32_t)((done >> 1) - 1) & 1u, ctrl, a.hdr);
        if (lane == 0) {
          const int cw = red.warp;
#pragma unroll
          for (int i = 0; i < 1 + 3 * PD; ++i) ctrl->endred[par][i * NCW + cw] = part[i];
          if (cw == 0) { ctrl->end_ce[par] = ce; ctrl->end_correct[par] = (a_own == y); }
          mbar_arrive(&ctrl->end_full[par]);
        }
      }
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
  const int64_t n_seg_max = dtype == CODISTILL_F32 ? max_row_segments<float>(a.row_stride, a.classes)
                                                   : max_row_segments<__nv_bfloat16>(a.row_stride, a.classes);
  // Two CTAs of 8 consumer warps per SM when the row buffer leaves room for a ring in half an SM's
  // shared memory, otherwise one CTA of 16 consumer warps.
  for (int pass = 0; pass < 2; ++pass) {
    TmaCfg c;
    c.consumer_warps = pass == 0 ? 8 : 16;
    c.ctas_per_sm = pass == 0 ? 2 : 1;
    c.chunk_bytes = (uint32_t)c.consumer_warps * 32u * kSegPerThread * 16u;
    const int64_t seg_per_chunk = c.chunk_bytes / 16;
    c.pieces = (int)((n_seg_max + seg_per_chunk - 1) / seg_per_chunk);
    if (c.pieces > kMaxPieces) continue;
    const int64_t own_buf = (int64_t)c.pieces * c.chunk_bytes;  // whole pieces, so that every piece has a home
    const int64_t per_cta = c.ctas_per_sm == 1 ? (int64_t)smem_optin : ((int64_t)smem_optin + 1024) / c.ctas_per_sm - 1024;
    int64_t st = (per_cta - kCtrlBytes - own_buf) / c.chunk_bytes;
    const int min_stages = a.n_peers > 0 ? (pass == 0 ? 4 : 2) : 0;
    if (st < min_stages) continue;
    if (st > kMaxStages) st = kMaxStages;
    if (a.n_peers == 0) st = 1;
    c.stages = (int)st;
    c.own_buf_bytes = (uint32_t)own_buf;
    c.smem_bytes = (uint32_t)(kCtrlBytes + own_buf + st * c.chunk_bytes);
    *out = c;
    return true;
  }
  return false;
}

bool tma_supported(const KArgs& a, int dtype, int smem_optin) {
  TmaCfg c;
  return tma_config(a, dtype, smem_optin, &c);
}

// CTAs per SM the staged kernel would run with (0: it does not take the call).
int tma_ctas_per_sm(const KArgs& a, int dtype, int smem_optin) {
  TmaCfg c;
  return tma_config(a, dtype, smem_optin, &c) ? c.ctas_per_sm : 0;
}

template <typename T, int P, bool PW, int NCW>
static cudaError_t launch_one(const KArgs& a, const TmaCfg& c, int grid, cudaStream_t stream) {
  cudaError_t e = cudaFuncSetAttribute(rows_tma_kernel<T, P, PW, NCW>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c.smem_bytes);
  if (e != cudaSuccess) return e;
  e = launch_overlapped(rows_tma_kernel<T, P, PW, NCW>, dim3(grid), dim3(NCW * 32 + kProducerThreads), c.smem_bytes, stream, a, c);
  return e != cudaSuccess ? e : cudaGetLastError();
}

template <typename T, int NCW>
static cudaError_t launch_peers(const KArgs& a, const TmaCfg& c, int grid, cudaStream_t stream) {
  const bool pw = a.peer_reduce == CODISTILL_PEERS_PAIRWISE_MEAN;  // with one peer both readings coincide
  switch (a.n_peers) {
    case 0: return launch_one<T, 0, true, NCW>(a, c, grid, stream);
    case 1: return launch_one<T, 1, true, NCW>(a, c, grid, stream);
    case 2: return pw ? launch_one<T, 2, true, NCW>(a, c, grid, stream) : launch_one<T, 2, false, NCW>(a, c, grid, stream);
    case 3: return pw ? launch_one<T, 3, true, NCW>(a, c, grid, stream) : launch_one<T, 3, false, NCW>(a, c, grid, stream);
    case 7: return pw ? launch_one<T, 7, true, NCW>(a, c, grid, stream) : launch_one<T, 7, false, NCW>(a, c, grid, stream);
    default: return cudaErrorNotSupported;
  }
}

template <typename T>
static cudaError_t launch_dtype(const KArgs& a, const TmaCfg& c, int grid, cudaStream_t stream) {
  return c.consumer_warps == 8 ? launch_peers<T, 8>(a, c, grid, stream) : launch_peers<T, 16>(a, c, grid, stream);
}

cudaError_t launch_tma(const KArgs& a, int dtype, int num_sms, int smem_optin, cudaStream_t stream) {
  TmaCfg c;
  if (!tma_config(a, dtype, smem_optin, &c)) return cudaErrorNotSupported;
  const int64_t rows = a.row_end - a.row_begin;
  if (rows <= 0) return cudaSuccess;
  const int64_t slots = (int64_t)num_sms * c.ctas_per_sm;
  const int grid = (int)(rows < slots ? rows : slots);
  return dtype == CODISTILL_F32 ? launch_dtype<float>(a, c, grid, stream) : launch_dtype<__nv_bfloat16>(a, c, grid, stream);
}

}  // namespace codistill
