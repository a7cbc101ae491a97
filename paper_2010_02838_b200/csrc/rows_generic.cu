// Generic row kernels: one warp per row ("warp" regime, short rows) or one CTA per row ("block"
// regime, any row length).  They read the logits straight from global memory (16-byte packets
// when the rows are 16-byte aligned, single elements otherwise), make one pass for the own-row
// statistics, one per peer where peer statistics are needed, and one element-wise pass that
// forms the distillation term and writes the gradient.  Every option of the objective of
// Algorithm 1 is served here; the TMA-staged kernel in rows_tma.cu covers long bf16/fp32 rows
// faster and falls back to these.
#include "common.cuh"

namespace codistill {

constexpr int kWarpRegimeThreads = 256;   // 8 rows per CTA
constexpr int kBlockRegimeThreads = 512;

struct PeerStats {       // per-peer row statistics kept in shared memory (KL forms)
  float max_v[kMaxPeers];
  float log_sum[kMaxPeers];
  float kl_rev[kMaxPeers];   // KL(p^T || t_j), the row constant in the reverse direction's gradient
};

template <typename T, int V, int G>
__device__ __forceinline__ void process_row(const KArgs& a, int64_t r, int lane, float w, float* scratch,
                                            PeerStats* ps) {
  const int64_t C = a.classes;
  const int64_t lr = r - a.row_begin;
  const T* __restrict__ z_row = reinterpret_cast<const T*>(a.own) + lr * a.row_stride;
  T* __restrict__ g_row = a.grad ? reinterpret_cast<T*>(a.grad) + lr * a.row_stride : nullptr;
  const int P = a.n_peers;
  const int64_t n_packets = (C + V - 1) / V;

  if (!row_valid(a, r)) {  // masked: zero gradient row, no loss, no counts
    if (g_row) {
      float zero[V];
#pragma unroll
      for (int i = 0; i < V; ++i) zero[i] = 0.f;
      for (int64_t k = lane; k < n_packets; k += G) {
        const int64_t c = k * V;
        store_packet<T, V>(g_row, c, zero, (int)min((int64_t)V, C - c));
      }
    }
    if (lane == 0) { a.row_loss[r] = 0.f; a.row_flags[r] = 0u; }
    return;
  }
  const int y = a.labels[r];
  // the softmax-KL family: peer as target (forward), own as target (reverse), or half of each (symmetric)
  const bool kl = a.dist == CODISTILL_DIST_KL_SOFTMAX || a.dist == CODISTILL_DIST_KL_REVERSE || a.dist == CODISTILL_DIST_KL_SYMMETRIC;
  const float wf = a.dist == CODISTILL_DIST_KL_SOFTMAX ? 1.f : a.dist == CODISTILL_DIST_KL_SYMMETRIC ? 0.5f : 0.f;
  const float wr = a.dist == CODISTILL_DIST_KL_REVERSE ? 1.f : a.dist == CODISTILL_DIST_KL_SYMMETRIC ? 0.5f : 0.f;
  const bool centred = (a.dist == CODISTILL_DIST_MSE_CENTRED);  // MSE between logits centred on their class means
  const bool with_term = (P >= 1 && a.alpha != 0.f);
  const float inv_T = 1.f / a.temperature;

  // ---- own row: max and first arg-max
  float best = -INFINITY;
  int best_i = 0x7fffffff;
  for (int64_t k = lane; k < n_packets; k += G) {
    float v[V];
    load_packet<T, V>(z_row, k * V, v);
#pragma unroll
    for (int i = 0; i < V; ++i) {
      const int64_t c = k * V + i;
      if (c < C && v[i] > best) { best = v[i]; best_i = (int)c; }
    }
  }
  Group<G>::argmax(best, best_i, scratch);
  const float m = best;
  const int a_own = best_i;

  // ---- own row: sum exp(z - m), sum z, sum exp((z - m)/T)
  float acc[3] = {0.f, 0.f, 0.f};
  for (int64_t k = lane; k < n_packets; k += G) {
    float v[V];
    load_packet<T, V>(z_row, k * V, v);
#pragma unroll
    for (int i = 0; i < V; ++i) {
      if (k * V + i < C) {
        acc[0] += expf(v[i] - m);
        acc[1] += v[i];
        if (kl) acc[2] += expf((v[i] - m) * inv_T);
      }
    }
  }
  Group<G>::sum(acc, scratch);
  const float S = acc[0], sum_z = acc[1];
  const float log_ST = kl ? logf(acc[2]) : 0.f;
  const float zy = Elem<T>::to_f32(z_row[y]);
  const float lse = m + logf(S);
  const float ce = lse - (1.f - a.eps) * zy - (a.eps / (float)C) * sum_z;

  // ---- peers: arg-max agreement and (KL, pairwise) softmax statistics
  uint32_t flags = (a_own == y) ? 1u : 0u;
  const bool peer_stats = with_term && kl && a.peer_reduce == CODISTILL_PEERS_PAIRWISE_MEAN;
  const bool peer_means = with_term && centred;
  if (P >= 1 && (a.want_flags || peer_stats || peer_means)) {
    for (int j = 0; j < P; ++j) {
      const T* __restrict__ p_row = reinterpret_cast<const T*>(a.peers[j]) + lr * a.row_stride;
      float pb = -INFINITY;
      int pi = 0x7fffffff;
      for (int64_t k = lane; k < n_packets; k += G) {
        float v[V];
        load_packet<T, V>(p_row, k * V, v);
#pragma unroll
        for (int i = 0; i < V; ++i) {
          const int64_t c = k * V + i;
          if (c < C && v[i] > pb) { pb = v[i]; pi = (int)c; }
        }
      }
      Group<G>::argmax(pb, pi, scratch);
      if (pi == a_own) flags |= (2u << j);
      if (peer_means) {  // difference of the class means: (mean z) - (mean z^(j)), the shift the centring removes
        float sv[1] = {0.f};
        for (int64_t k = lane; k < n_packets; k += G) {
          float v[V];
          load_packet<T, V>(p_row, k * V, v);
#pragma unroll
          for (int i = 0; i < V; ++i)
            if (k * V + i < C) sv[0] += v[i];
        }
        Group<G>::sum(sv, scratch);
        if (lane == 0) ps->max_v[j] = (sum_z - sv[0]) / (float)C;
      }
      if (peer_stats) {
        float sj[1] = {0.f};
        for (int64_t k = lane; k < n_packets; k += G) {
          float v[V];
          load_packet<T, V>(p_row, k * V, v);
#pragma unroll
          for (int i = 0; i < V; ++i)
            if (k * V + i < C) sj[0] += expf((v[i] - pb) * inv_T);
        }
        Group<G>::sum(sj, scratch);
        const float lsj = logf(sj[0]);
        if (lane == 0) { ps->max_v[j] = pb; ps->log_sum[j] = lsj; }
        if (wr != 0.f) {   // KL(p^T || t_j) = sum_c p^T_c (log p^T_c - log t_jc)
          float kj[1] = {0.f};
          for (int64_t k = lane; k < n_packets; k += G) {
            float v[V], o[V];
            load_packet<T, V>(p_row, k * V, v);
            load_packet<T, V>(z_row, k * V, o);
#pragma unroll
            for (int i = 0; i < V; ++i) {
              if (k * V + i < C) {
                // log p - log t with the large parts cancelled before they are rounded
                const float log_p = (o[i] - m) * inv_T - log_ST;
                const float diff = ((o[i] - v[i]) - (m - pb)) * inv_T - (log_ST - lsj);
                kj[0] = fmaf(expf(log_p), diff, kj[0]);
              }
            }
          }
          Group<G>::sum(kj, scratch);
          if (lane == 0) ps->kl_rev[j] = kj[0];
        }
      }
    }
    if (peer_stats || peer_means) {
      if constexpr (G > 32) __syncthreads(); else __syncwarp();
    }
  }

  // ---- KL against the averaged peer: statistics of zbar / T
  float mb = 0.f, log_Sb = 0.f, kl_rev_b = 0.f;
  const float inv_P = P >= 1 ? 1.f / (float)P : 0.f;
  if (with_term && kl && a.peer_reduce == CODISTILL_PEERS_MEAN_TARGET) {
    float bm = -INFINITY;
    for (int64_t k = lane; k < n_packets; k += G) {
      float zb[V];
#pragma unroll
      for (int i = 0; i < V; ++i) zb[i] = 0.f;
      for (int j = 0; j < P; ++j) {
        float v[V];
        load_packet<T, V>(reinterpret_cast<const T*>(a.peers[j]) + lr * a.row_stride, k * V, v);
#pragma unroll
        for (int i = 0; i < V; ++i) zb[i] += v[i];
      }
#pragma unroll
      for (int i = 0; i < V; ++i)
        if (k * V + i < C) bm = fmaxf(bm, zb[i] * inv_P);
    }
    mb = Group<G>::max(bm, scratch);
    float sb[1] = {0.f};
    for (int64_t k = lane; k < n_packets; k += G) {
      float zb[V];
#pragma unroll
      for (int i = 0; i < V; ++i) zb[i] = 0.f;
      for (int j = 0; j < P; ++j) {
        float v[V];
        load_packet<T, V>(reinterpret_cast<const T*>(a.peers[j]) + lr * a.row_stride, k * V, v);
#pragma unroll
        for (int i = 0; i < V; ++i) zb[i] += v[i];
      }
#pragma unroll
      for (int i = 0; i < V; ++i)
        if (k * V + i < C) sb[0] += expf((zb[i] * inv_P - mb) * inv_T);
    }
    Group<G>::sum(sb, scratch);
    log_Sb = logf(sb[0]);
    if (wr != 0.f) {   // KL(p^T || t) against the softmax of the averaged peers
      float kb[1] = {0.f};
      for (int64_t k = lane; k < n_packets; k += G) {
        float zb[V], o[V];
#pragma unroll
        for (int i = 0; i < V; ++i) zb[i] = 0.f;
        for (int j = 0; j < P; ++j) {
          float v[V];
          load_packet<T, V>(reinterpret_cast<const T*>(a.peers[j]) + lr * a.row_stride, k * V, v);
#pragma unroll
          for (int i = 0; i < V; ++i) zb[i] += v[i];
        }
        load_packet<T, V>(z_row, k * V, o);
#pragma unroll
        for (int i = 0; i < V; ++i) {
          if (k * V + i < C) {
            const float log_p = (o[i] - m) * inv_T - log_ST;
            const float diff = ((o[i] - zb[i] * inv_P) - (m - mb)) * inv_T - (log_ST - log_Sb);
            kb[0] = fmaf(expf(log_p), diff, kb[0]);
          }
        }
      }
      Group<G>::sum(kb, scratch);
      kl_rev_b = kb[0];
    }
  }

  // ---- element-wise pass: distillation term and gradient
  const float inv_S = 1.f / S;
  const float q_off = a.eps / (float)C;
  const float two_over_C = 2.f / (float)C;
  const float temp = a.temperature;
  float dacc[1] = {0.f};  // sum over classes of the distance integrand
  if (with_term || g_row) {
    for (int64_t k = lane; k < n_packets; k += G) {
      const int64_t c0 = k * V;
      float v[V], dD[V], g[V];
      load_packet<T, V>(z_row, c0, v);
#pragma unroll
      for (int i = 0; i < V; ++i) dD[i] = 0.f;
      if (with_term) {
        if (!kl) {
          float sd[V], sq[V];
#pragma unroll
          for (int i = 0; i < V; ++i) { sd[i] = 0.f; sq[i] = 0.f; }
          for (int j = 0; j < P; ++j) {
            float u[V];
            load_packet<T, V>(reinterpret_cast<const T*>(a.peers[j]) + lr * a.row_stride, c0, u);
            const float shift = centred ? ps->max_v[j] : 0.f;
#pragma unroll
            for (int i = 0; i < V; ++i) {
              const float d = (v[i] - u[i]) - shift;
              sd[i] += d;
              sq[i] = fmaf(d, d, sq[i]);
            }
          }
#pragma unroll
          for (int i = 0; i < V; ++i) {
            const float dbar = sd[i] * inv_P;  // z_c - zbar_c
            dD[i] = two_over_C * dbar;
            if (c0 + i < C)
              dacc[0] += (a.peer_reduce == CODISTILL_PEERS_PAIRWISE_MEAN) ? sq[i] * inv_P : dbar * dbar;
          }
        } else {
          float log_pT[V], pT[V];
#pragma unroll
          for (int i = 0; i < V; ++i) {
            log_pT[i] = (v[i] - m) * inv_T - log_ST;
            pT[i] = expf(log_pT[i]);
          }
          if (a.peer_reduce == CODISTILL_PEERS_PAIRWISE_MEAN) {
            float tbar[V];
#pragma unroll
            for (int i = 0; i < V; ++i) tbar[i] = 0.f;
            for (int j = 0; j < P; ++j) {
              float u[V];
              load_packet<T, V>(reinterpret_cast<const T*>(a.peers[j]) + lr * a.row_stride, c0, u);
              const float mj = ps->max_v[j], lsj = ps->log_sum[j], kj = wr != 0.f ? ps->kl_rev[j] : 0.f;   // unset without a reverse part
#pragma unroll
              for (int i = 0; i < V; ++i) {
                const float log_t = (u[i] - mj) * inv_T - lsj;
                const float t = expf(log_t);
                const float diff = ((v[i] - u[i]) - (m - mj)) * inv_T - (log_ST - lsj);   // log p - log t, large parts cancelled first
                // forward: t (log t - log p), derivative T (p - t); reverse: p (log p - log t), derivative T p (diff - KL_j)
                tbar[i] += wf * (pT[i] - t) + wr * pT[i] * (diff - kj);
                if (c0 + i < C) dacc[0] += wr * pT[i] * diff - wf * t * diff;
              }
            }
#pragma unroll
            for (int i = 0; i < V; ++i) dD[i] = temp * tbar[i] * inv_P;
          } else {
            float zb[V];
#pragma unroll
            for (int i = 0; i < V; ++i) zb[i] = 0.f;
            for (int j = 0; j < P; ++j) {
              float u[V];
              load_packet<T, V>(reinterpret_cast<const T*>(a.peers[j]) + lr * a.row_stride, c0, u);
#pragma unroll
              for (int i = 0; i < V; ++i) zb[i] += u[i];
            }
#pragma unroll
            for (int i = 0; i < V; ++i) {
              const float log_t = (zb[i] * inv_P - mb) * inv_T - log_Sb;
              const float t = expf(log_t);
              const float diff = ((v[i] - zb[i] * inv_P) - (m - mb)) * inv_T - (log_ST - log_Sb);
              if (c0 + i < C) dacc[0] += wr * pT[i] * diff - wf * t * diff;
              dD[i] = temp * (wf * (pT[i] - t) + wr * pT[i] * (diff - kl_rev_b));
            }
          }
        }
      }
      if (g_row) {
#pragma unroll
        for (int i = 0; i < V; ++i) {
          const float p = expf(v[i] - m) * inv_S;
          const float q = q_off + ((c0 + i == (int64_t)y) ? (1.f - a.eps) : 0.f);
          g[i] = w * ((p - q) + a.alpha * dD[i]);
        }
        store_packet<T, V>(g_row, c0, g, (int)min((int64_t)V, C - c0));
      }
    }
  }
  float D = 0.f;
  if (with_term) {
    Group<G>::sum(dacc, scratch);
    if (!kl) D = dacc[0] / (float)C;
    else D = temp * temp * dacc[0] * (a.peer_reduce == CODISTILL_PEERS_PAIRWISE_MEAN ? inv_P : 1.f);
  }
  if (lane == 0) {
    a.row_loss[r] = with_term ? fmaf(a.alpha, D, ce) : ce;
    a.row_flags[r] = flags;
  }
}

template <typename T, int V, int G>
__global__ void __launch_bounds__(G == 32 ? kWarpRegimeThreads : kBlockRegimeThreads)
rows_generic_kernel(const __grid_constant__ KArgs a) {
  __shared__ float scratch[4 * 33];
  __shared__ PeerStats peer_stats[G == 32 ? kWarpRegimeThreads / 32 : 1];
  __shared__ double sh_final[32];
  __shared__ int sh_flag;

  wait_for_prior_grid();
  float w = 1.f;
  if (a.reduction == CODISTILL_REDUCE_MEAN_VALID) {
    const int64_t nv = total_valid(a);
    w = 1.f / (float)(nv > 1 ? nv : 1);
  }
  if constexpr (G == 32) {
    const int warps_per_cta = kWarpRegimeThreads / 32;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int64_t r = a.row_begin + (int64_t)blockIdx.x * warps_per_cta + warp; r < a.row_end;
         r += (int64_t)gridDim.x * warps_per_cta)
      process_row<T, V, 32>(a, r, lane, w, nullptr, &peer_stats[warp]);
  } else {
    for (int64_t r = a.row_begin + blockIdx.x; r < a.row_end; r += gridDim.x)
      process_row<T, V, G>(a, r, threadIdx.x, w, scratch, &peer_stats[0]);
  }
  finish_cta(a, sh_final, &sh_flag);
}

// Host side: pick the instantiation and launch.  `vec` says the rows are 16-byte aligned.
cudaError_t launch_generic(const KArgs& a, int dtype, bool warp_regime, bool vec, int num_sms, cudaStream_t stream) {
  const int64_t rows = a.row_end - a.row_begin;
  if (rows <= 0) return cudaSuccess;
  int64_t grid;
  int threads;
  if (warp_regime) {
    threads = kWarpRegimeThreads;
    const int64_t ctas = (rows + (kWarpRegimeThreads / 32) - 1) / (kWarpRegimeThreads / 32);
    grid = ctas < (int64_t)num_sms * 8 ? ctas : (int64_t)num_sms * 8;
  } else {
    threads = kBlockRegimeThreads;
    grid = rows < (int64_t)num_sms * 4 ? rows : (int64_t)num_sms * 4;
  }
  cudaError_t err = cudaSuccess;
#define CODISTILL_LAUNCH(T, V, G) err = launch_overlapped(rows_generic_kernel<T, V, G>, dim3((unsigned)grid), dim3(threads), 0, stream, a)
  if (dtype == CODISTILL_F32) {
    if (warp_regime) { if (vec) CODISTILL_LAUNCH(float, 4, 32); else CODISTILL_LAUNCH(float, 1, 32); }
    else { if (vec) CODISTILL_LAUNCH(float, 4, kBlockRegimeThreads); else CODISTILL_LAUNCH(float, 1, kBlockRegimeThreads); }
  } else {
    if (warp_regime) { if (vec) CODISTILL_LAUNCH(__nv_bfloat16, 8, 32); else CODISTILL_LAUNCH(__nv_bfloat16, 1, 32); }
    else { if (vec) CODISTILL_LAUNCH(__nv_bfloat16, 8, kBlockRegimeThreads); else CODISTILL_LAUNCH(__nv_bfloat16, 1, kBlockRegimeThreads); }
  }
#undef CODISTILL_LAUNCH
  return err != cudaSuccess ? err : cudaGetLastError();
}

}  // namespace codistill
