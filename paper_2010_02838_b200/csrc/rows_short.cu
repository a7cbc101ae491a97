// Short rows in one launch ("short" regime): rows of up to 1024 classes, MSE-on-logits distance, up to 7 peers.
//
// One warp per row, the own row held in registers from its single read: maximum and first arg-max, sum exp and
// sum z come from the registers, then the peers are read once each (differences against the registers,
// squared distance, their arg-maxes), and the gradient is formed from the registers and written.  Problems of
// this size fit the L2 cache and are bound by launch latency, so the whole call is a single cooperative
// launch: every CTA counts the valid rows of the (short) mask itself instead of waiting for a counting kernel,
// and after a grid-wide barrier CTA 0 sums the per-row losses in a fixed order and counts the flag bits.
#include <cooperative_groups.h>

#include "common.cuh"

namespace cg = cooperative_groups;

namespace codistill {

constexpr int kShortThreads = 256;          // 8 rows per CTA at a time
constexpr int kShortMaxClasses = 1024;      // 32 lanes x 32 values held per lane
constexpr int kShortMaxPeers = 7;
constexpr int64_t kShortMaxRows = 16384;    // every CTA scans the whole mask: keep it cheap

// T: element type; V: elements per load (1, or a 16-byte packet); NPK: loads per lane that cover a row.
template <typename T, int V, int NPK>
__global__ void __launch_bounds__(kShortThreads) rows_short_kernel(const __grid_constant__ KArgs a) {
  constexpr int NE = V * NPK;               // values per lane
  __shared__ long long sh_cnt[2][kShortThreads / 32];
  __shared__ int sh_bad;
  __shared__ double sh_fin[32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t C = a.classes, R = a.rows_total;
  const int P = a.n_peers;
  const bool with_term = (P >= 1 && a.alpha != 0.f);

  // ---- valid / masked rows of the whole call, counted by every CTA (fixed order: the result is the same everywhere)
  long long valid = 0, masked = 0;
  int bad = 0;
  for (int64_t r = tid; r < R; r += kShortThreads) {
    const bool on = (a.mask == nullptr) || a.mask[r] != 0;
    const int32_t y = a.labels[r];
    const bool ok = y >= 0 && (int64_t)y < C;
    if (on && ok) ++valid; else ++masked;
    bad |= (on && !ok);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    valid += __shfl_xor_sync(0xffffffffu, valid, o);
    masked += __shfl_xor_sync(0xffffffffu, masked, o);
  }
  if (tid == 0) sh_bad = 0;
  __syncthreads();
  if (bad) sh_bad = 1;
  if (lane == 0) { sh_cnt[0][warp] = valid; sh_cnt[1][warp] = masked; }
  __syncthreads();
  long long n_valid = 0, n_masked = 0;
#pragma unroll
  for (int k = 0; k < kShortThreads / 32; ++k) { n_valid += sh_cnt[0][k]; n_masked += sh_cnt[1][k]; }
  const float w = a.reduction == CODISTILL_REDUCE_MEAN_VALID ? 1.f / (float)(n_valid > 1 ? n_valid : 1) : 1.f;
  const float inv_C = 1.f / (float)C;
  const float inv_P = P >= 1 ? 1.f / (float)P : 0.f;
  const float cd = with_term ? w * a.alpha * (2.f * inv_C) * inv_P : 0.f;   // sum_j (z - z_j) -> w alpha dD/dz
  const float cq = w * a.eps * inv_C, cy = w * (1.f - a.eps);
  const bool pairwise = a.peer_reduce == CODISTILL_PEERS_PAIRWISE_MEAN;

  // ---- rows: one warp each
  const int warps_per_cta = kShortThreads / 32;
  for (int64_t r = a.row_begin + (int64_t)blockIdx.x * warps_per_cta + warp; r < a.row_end; r += (int64_t)gridDim.x * warps_per_cta) {
    const int64_t lr = r - a.row_begin;
    const T* __restrict__ z_row = reinterpret_cast<const T*>(a.own) + lr * a.row_stride;
    T* __restrict__ g_row = a.grad ? reinterpret_cast<T*>(a.grad) + lr * a.row_stride : nullptr;
    const int32_t y = a.labels[r];
    const bool row_ok = (a.mask == nullptr || a.mask[r] != 0) && y >= 0 && (int64_t)y < C;
    if (!row_ok) {   // masked: zero gradient row, no loss, no counts
      if (g_row) {
        float zero[V];
#pragma unroll
        for (int i = 0; i < V; ++i) zero[i] = 0.f;
#pragma unroll
        for (int k = 0; k < NPK; ++k) {
          const int64_t c = ((int64_t)k * 32 + lane) * V;
          if (c < C) store_packet<T, V>(g_row, c, zero, (int)min((int64_t)V, C - c));
        }
      }
      if (lane == 0) { a.row_loss[r] = 0.f; a.row_flags[r] = 0u; }
      continue;
    }
    // own row into registers; columns past the row read as -inf (no maximum, exp = 0) and are never stored
    float z[NE];
#pragma unroll
    for (int k = 0; k < NPK; ++k) {
      const int64_t c = ((int64_t)k * 32 + lane) * V;
      float v[V];
#pragma unroll
      for (int i = 0; i < V; ++i) v[i] = -INFINITY;
      if (c + V <= C) {
        load_packet<T, V>(z_row, c, v);
      } else if (c < C) {
#pragma unroll
        for (int i = 0; i < V; ++i)
          if (c + i < C) v[i] = Elem<T>::to_f32(z_row[c + i]);
      }
#pragma unroll
      for (int i = 0; i < V; ++i) z[k * V + i] = v[i];
    }
    float best = -INFINITY;
    int best_i = 0x7fffffff;
#pragma unroll
    for (int e = 0; e < NE; ++e) {
      const int c = ((e / V) * 32 + lane) * V + (e % V);
      if (z[e] > best) { best = z[e]; best_i = c; }   // a lane's columns rise with e: strict '>' keeps its first
    }
    warp_argmax(best, best_i);
    const float m = best;
    const int a_own = best_i;
    float S = 0.f, sum_z = 0.f;
#pragma unroll
    for (int e = 0; e < NE; ++e) {
      S += expf(z[e] - m);                          // exp(-inf) = 0 for the columns past the row
      sum_z += z[e] == -INFINITY ? 0.f : z[e];
    }
    S = warp_sum(S);
    sum_z = warp_sum(sum_z);
    float zy;
    {
      // the label's logit sits in one lane's registers: pick it with compile-time indices, hand it to all
      float mine = 0.f;
#pragma unroll
      for (int e = 0; e < NE; ++e) {
        const int c = ((e / V) * 32 + lane) * V + (e % V);
        if (c == y) mine = z[e];
      }
      zy = warp_sum(mine);
    }
    const float ce = (m + logf(S)) - (1.f - a.eps) * zy - (a.eps * inv_C) * sum_z;

    // peers: each read once; sd = sum_j (z - z_j) per column, the squared distance, the peers' first arg-maxes
    float sd[NE];
#pragma unroll
    for (int e = 0; e < NE; ++e) sd[e] = 0.f;
    float dist = 0.f;
    uint32_t flags = (a_own == y) ? 1u : 0u;
    if (P >= 1 && (with_term || a.want_flags)) {
      for (int j = 0; j < P; ++j) {
        const T* __restrict__ p_row = reinterpret_cast<const T*>(a.peers[j]) + lr * a.row_stride;
        float pv[NE];
#pragma unroll
        for (int k = 0; k < NPK; ++k) {
          const int64_t c = ((int64_t)k * 32 + lane) * V;
          float v[V];
#pragma unroll
          for (int i = 0; i < V; ++i) v[i] = -INFINITY;
          if (c + V <= C) {
            load_packet<T, V>(p_row, c, v);
          } else if (c < C) {
#pragma unroll
            for (int i = 0; i < V; ++i)
              if (c + i < C) v[i] = Elem<T>::to_f32(p_row[c + i]);
          }
#pragma unroll
          for (int i = 0; i < V; ++i) pv[k * V + i] = v[i];
        }
        float pb = -INFINITY;
        int pi = 0x7fffffff;
#pragma unroll
        for (int e = 0; e < NE; ++e) {
          const int c = ((e / V) * 32 + lane) * V + (e % V);
          if (pv[e] > pb) { pb = pv[e]; pi = c; }
          const float d = z[e] == -INFINITY ? 0.f : z[e] - pv[e];
          sd[e] += d;
          if (pairwise) dist = fmaf(d, d, dist);
        }
        warp_argmax(pb, pi);
        if (pi == a_own) flags |= (2u << j);
      }
      if (!pairwise) {
#pragma unroll
        for (int e = 0; e < NE; ++e) dist = fmaf(sd[e], sd[e], dist);   // (sum_j d)^2, scaled by 1/P^2 below
      }
      dist = warp_sum(dist);
    }
    if (g_row) {
      const float cp = w / S;
#pragma unroll
      for (int k = 0; k < NPK; ++k) {
        const int64_t c = ((int64_t)k * 32 + lane) * V;
        if (c < C) {
          float g[V];
#pragma unroll
          for (int i = 0; i < V; ++i) {
            const float gv = fmaf(expf(z[k * V + i] - m), cp, fmaf(sd[k * V + i], cd, -cq));
            g[i] = (c + i == (int64_t)y) ? gv - cy : gv;
          }
          store_packet<T, V>(g_row, c, g, (int)min((int64_t)V, C - c));
        }
      }
    }
    if (lane == 0) {
      float D = 0.f;
      if (with_term) D = pairwise ? dist * inv_P * inv_C : dist * inv_P * inv_P * inv_C;
      a.row_loss[r] = with_term ? fmaf(a.alpha, D, ce) : ce;
      a.row_flags[r] = flags;
    }
  }

  // ---- every row is written: CTA 0 sums the losses in a fixed order and counts the flag bits
  __threadfence();
  cg::this_grid().sync();
  if (blockIdx.x != 0) return;
  const int nw = kShortThreads / 32;
  double s = 0.0;
  for (int64_t r = tid; r < R; r += kShortThreads) s += (double)__ldcg(a.row_loss + r);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_down_sync(0xffffffffu, s, o);
  if (lane == 0) sh_fin[warp] = s;
  __syncthreads();
  if (tid == 0) {
    double total = 0.0;
    for (int k = 0; k < nw; ++k) total += sh_fin[k];
    if (a.reduction == CODISTILL_REDUCE_MEAN_VALID) total /= (double)(n_valid > 1 ? n_valid : 1);
    *a.reduced_loss = (float)total;
    if (a.dev_status) *a.dev_status = sh_bad ? CODISTILL_DEV_BAD_LABEL : 0;
    if (a.counters) { a.counters[0] = n_valid; a.counters[1] = n_masked; }
  }
  if (a.counters) {
    long long* shi = reinterpret_cast<long long*>(sh_fin);
    for (int bit = 0; bit <= P; ++bit) {
      long long cnt = 0;
      for (int64_t r = tid; r < R; r += kShortThreads) cnt += (__ldcg(a.row_flags + r) >> bit) & 1u;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) cnt += __shfl_down_sync(0xffffffffu, cnt, o);
      __syncthreads();
      if (lane == 0) shi[warp] = cnt;
      __syncthreads();
      if (tid == 0) {
        long long total = 0;
        for (int k = 0; k < nw; ++k) total += shi[k];
        a.counters[2 + bit] = total;
      }
    }
  }
}

// ------------------------------------------------------------------ host side
// The call as a whole (the launch does its own counting and final reduction): rows [0, rows_total) of `a`.
bool short_supported(const KArgs& a, int dtype) {
  if (a.dist != CODISTILL_DIST_MSE_LOGITS || a.n_peers > kShortMaxPeers) return false;
  if (a.classes > kShortMaxClasses || a.rows_total > kShortMaxRows || a.rows_total < 1) return false;
  if (a.row_begin != 0 || a.row_end != a.rows_total || !a.fused_finalize) return false;
  (void)dtype;
  return true;
}

template <typename T, int V, int NPK>
static cudaError_t short_launch_one(const KArgs& a, int num_sms, cudaStream_t stream) {
  auto kernel = rows_short_kernel<T, V, NPK>;
  static int per_sm[64];   // co-resident CTAs per SM, asked once per device (0: not asked yet; benign if asked twice)
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  int occ = (dev >= 0 && dev < 64) ? per_sm[dev] : 0;
  if (occ == 0) {
    if ((e = cuda_note(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kernel, kShortThreads, 0), "cudaOccupancyMaxActiveBlocksPerMultiprocessor")) != cudaSuccess) return e;
    if (occ < 1) return cuda_note(cudaErrorLaunchOutOfResources, "short-row kernel does not fit an SM");
    if (dev >= 0 && dev < 64) per_sm[dev] = occ;
  }
  const int64_t ctas = (a.rows_total + (kShortThreads / 32) - 1) / (kShortThreads / 32);
  const int64_t cap = (int64_t)num_sms * occ;
  const unsigned grid = (unsigned)(ctas < cap ? ctas : cap);
  KArgs args = a;
  void* params[] = {&args};
  e = cuda_note(cudaLaunchCooperativeKernel(reinterpret_cast<void*>(kernel), dim3(grid), dim3(kShortThreads), params, 0, stream),
                "cudaLaunchCooperativeKernel (short-row kernel)");
  return e != cudaSuccess ? e : cudaGetLastError();
}

template <typename T, int V>
static cudaError_t short_launch_v(const KArgs& a, int num_sms, cudaStream_t stream) {
  const int64_t per_lane = (a.classes + 32 * V - 1) / (32 * V);   // loads per lane that cover the row
  if (per_lane <= 1) return short_launch_one<T, V, 1>(a, num_sms, stream);
  if (per_lane <= 2) return short_launch_one<T, V, 2>(a, num_sms, stream);
  if (per_lane <= 4) return short_launch_one<T, V, 4>(a, num_sms, stream);
  if constexpr (V <= 4) {
    if (per_lane <= 8) return short_launch_one<T, V, 8>(a, num_sms, stream);
  }
  if constexpr (V == 1) {
    if (per_lane <= 16) return short_launch_one<T, V, 16>(a, num_sms, stream);
    if (per_lane <= 32) return short_launch_one<T, V, 32>(a, num_sms, stream);
  }
  return cudaErrorNotSupported;
}

// `vec`: rows and bases are 16-byte aligned (16-byte loads and stores), else element by element.
cudaError_t launch_short(const KArgs& a, int dtype, bool vec, int num_sms, cudaStream_t stream) {
  if (dtype == CODISTILL_F32) return vec ? short_launch_v<float, 4>(a, num_sms, stream) : short_launch_v<float, 1>(a, num_sms, stream);
  return vec ? short_launch_v<__nv_bfloat16, 8>(a, num_sms, stream) : short_launch_v<__nv_bfloat16, 1>(a, num_sms, stream);
}

}  // namespace codistill
