// Direct-load kernel for long rows, softmax-KL distance (the form Section 2 attributes to earlier
// work):  D = T^2 / (n-1) * sum_j KL(softmax(z_j / T) || softmax(z / T))   (pairwise), or
//         D = T^2 * KL(softmax(zbar / T) || softmax(z / T)), zbar the mean of the peer logits.
// Same organisation as rows_stream.cu (one CTA per row, nothing staged, 16-byte loads), with one
// more pass, because the peers' softmax statistics must be known before the gradient:
//   pass A   own row: maximum with first arg-max, sum exp(z - m), sum exp((z - m) / T), sum z;
//   pass A2  peer rows: per peer the maximum and sum exp((v - m_j) / T)   (mean target: of zbar);
//   pass B   own and peer rows again: t = softmax(peer / T), p^T = softmax(z / T), the distance
//            sum t (log t - log p^T), the gradient w [(p - q) + alpha T (p^T - mean_j t_j)].
// The second reads come shortly after the first ones and are largely served by L2.
// Arithmetic is carried in "exp units" U: natural logarithms for fp32 logits (expf / logf), base-2
// for bf16 logits (the hardware exp2); kU converts a natural-log quantity to U.
#include <type_traits>

#include "stream_common.cuh"

namespace codistill {

struct StreamKlShared {
  float4 red[2][kStreamMaxWarps];        // pass A: max, first segment, sum exp, sum z
  float red_t[2][kStreamMaxWarps];       // pass A: sum exp at temperature T
  float2 peer[2][kStreamMaxPeers][kStreamMaxWarps];  // pass A2: per peer (or mean target in slot 0): max, sum exp
  float endred[2][kStreamMaxWarps * (1 + 3 * kStreamMaxPeers)];
  long long next_row[2];
  double fin[32];
  int last_flag;
};

template <typename T> struct ExpUnits;
template <> struct ExpUnits<float> {
  static constexpr float kU = 1.f;
  __device__ static float ex(float x) { return expf(x); }
  __device__ static float lg(float x) { return logf(x); }
};
template <> struct ExpUnits<__nv_bfloat16> {
  static constexpr float kU = kLog2e;
  __device__ static float ex(float x) { return ex2_approx(x); }
  __device__ static float lg(float x) { return log2f(x); }
};

// exp_U of a pair whose arguments are already in U
template <typename T>
__device__ __forceinline__ float2 ex_pair(float2 x) { return make_float2(ExpUnits<T>::ex(x.x), ExpUnits<T>::ex(x.y)); }
__device__ __forceinline__ float2 pair_of(float v) { return make_float2(v, v); }

// CTAs per SM: with many peers three instead of the MSE kernel's four -- 168 registers per thread and no spills
// instead of 128 with 500 bytes of them (workload 5: 7.25 -> 6.96 ms; two CTAs per SM: 9.0 ms).
__host__ __device__ constexpr int stream_kl_ctas_per_sm(int /*peers*/) { return 3; }

template <typename T, int P, bool PW>
__global__ void __launch_bounds__(stream_threads(P), stream_kl_ctas_per_sm(P)) rows_stream_kl_kernel(const __grid_constant__ KArgs a) {
  using EU = ExpUnits<T>;
  constexpr int V = SegOps<T>::V;
  constexpr int H = SegOps<T>::H;
  constexpr int PD = P > 0 ? P : 1;
  constexpr int NS = PW ? PD : 1;  // peer statistics kept: one per peer, or one for the mean target
  constexpr int NT = stream_threads(P);
  constexpr int NW = NT / 32;
  // L2 prefetch distances (up to three peers): one batch of the own row in pass A, two iterations of the
  // peers' segments in the peer-statistics pass; 12 % on 64 KiB rows with one peer.  Pass B reads from the L2.
  constexpr int kAheadA = P <= 3 ? 1 : 0, kAheadP = P <= 3 ? 2 : 0;
  __shared__ StreamKlShared sh;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t C = a.classes;
  const bool with_term = (P >= 1 && a.alpha != 0.f);
  const bool stream_peers = (P >= 1) && (with_term || a.want_flags);

  wait_for_prior_grid();  // from here on the workspace header and the valid-row counts are read
  const uint64_t pol_keep = make_policy_keep();
  float w = 1.f;
  if (a.reduction == CODISTILL_REDUCE_MEAN_VALID) {
    const int64_t nv = total_valid(a);
    w = 1.f / (float)(nv > 1 ? nv : 1);
  }
  const float inv_P = P >= 1 ? 1.f / (float)P : 0.f;
  const float inv_C = 1.f / (float)C;
  const float temp = a.temperature, inv_T = 1.f / a.temperature;
  const float k1 = EU::kU, kT = EU::kU * inv_T;  // logit -> exponent argument at temperature 1 / T
  const bool t_one = (a.temperature == 1.f);      // softmax(z / T) is softmax(z): its exponentials are shared

  stream_draw_row(&sh.next_row[0], a.hdr, a.row_begin, tid);
  __syncthreads();
  int v = 0;  // valid rows done by this CTA
  for (int it = 0;; ++it) {
    const long long r = sh.next_row[it & 1];
    if (r >= a.row_end) break;
    stream_draw_row(&sh.next_row[(it + 1) & 1], a.hdr, a.row_begin, tid);
    // The row view is spelled out here instead of taken from stream_row(): with seven peers this kernel ran
    // 18 % slower with the shared helper (same registers and spills, different schedule), so it keeps its own.
    const int64_t lr = r - a.row_begin;
    const RowGeom g = row_geom<T>(lr, a.row_stride, C);
    const int64_t row_off = lr * a.row_stride;  // in elements
    const T* __restrict__ z_row = reinterpret_cast<const T*>(a.own) + row_off;
    T* __restrict__ g_row = a.grad ? reinterpret_cast<T*>(a.grad) + row_off : nullptr;
    const uint4* __restrict__ z_img = reinterpret_cast<const uint4*>(z_row - g.head);
    uint4* __restrict__ g_img = g_row ? reinterpret_cast<uint4*>(g_row - g.head) : nullptr;
    const int n_int = g.seg_hi > g.seg_lo ? g.seg_hi - g.seg_lo : 0;    // segments wholly inside the row
    const int cnt = n_int > tid ? (n_int - tid + NT - 1) / NT : 0;     // of which this thread has cnt: seg_lo + tid + NT * i
    const int s0 = g.seg_lo + tid;
    const bool edge_head = (tid == 0) && g.seg_lo > 0;
    const bool edge_tail = (tid == 32) && g.seg_hi < g.n_seg && (g.n_seg > 1 || g.seg_lo == 0);
    const bool edge = edge_head || edge_tail;
    const int edge_seg = edge_head ? 0 : g.n_seg - 1;
    const int y = a.labels[r];
    const bool valid = (a.mask == nullptr || a.mask[r] != 0) && y >= 0 && (int64_t)y < C;

    if (!valid) {  // masked row: zero gradient, no loss, no counts; nothing is read
      if (g_img) {
        for (int i = 0; i < cnt; ++i) g_img[s0 + i * NT] = make_uint4(0u, 0u, 0u, 0u);
        if (edge) {
#pragma unroll
          for (int i = 0; i < V; ++i) {
            const int64_t c = (int64_t)edge_seg * V - g.head + i;
            if (c >= 0 && c < C) g_row[c] = Elem<T>::from_f32(0.f);
          }
        }
      }
      if (tid == 0) { a.row_loss[r] = 0.f; a.row_flags[r] = 0u; }
      __syncthreads();  // orders the row-id hand-over
      continue;
    }
    const int par = v & 1;
    const T* p_row[PD];
    const uint4* p_img[PD];
#pragma unroll
    for (int j = 0; j < PD; ++j) {
      p_row[j] = P > 0 ? reinterpret_cast<const T*>(a.peers[j]) + row_off : nullptr;
      p_img[j] = P > 0 ? reinterpret_cast<const uint4*>(p_row[j] - g.head) : nullptr;
    }

    // ================= pass A: own-row statistics (online softmax at temperatures 1 and T)
    float best = -3.0e38f;  // finite, so that the first rescale is exp(-huge) = 0 and never NaN
    int best_seg = 0x7fffffff;
    float s_1 = 0.f, s_T = 0.f, z_sum = 0.f;
    auto own_values = [&](const float (&zv)[V], int s) {  // zv: values of one segment, -inf outside the row
      float fm = zv[0];
#pragma unroll
      for (int i = 1; i < V; ++i) fm = fmaxf(fm, zv[i]);
      const float old = best;
      if (fm > best || (fm == best && s < best_seg)) { best = fm; best_seg = s; }
      s_1 *= EU::ex((old - best) * k1);
      s_T *= EU::ex((old - best) * kT);
#pragma unroll
      for (int i = 0; i < V; ++i) {
        if (zv[i] != -INFINITY) {
          s_1 += EU::ex((zv[i] - best) * k1);
          s_T += EU::ex((zv[i] - best) * kT);
          z_sum += zv[i];
        }
      }
    };
    {
      // segments wholly inside the row: packed pairs, several loads in flight; sums relative to the running maximum
      float2 s1p = make_float2(0.f, 0.f), sTp = make_float2(0.f, 0.f), zsp = make_float2(0.f, 0.f);
      const float2 k1_2 = pair_of(k1), kT_2 = pair_of(kT);
      for (int i0 = 0; i0 < cnt; i0 += kBatchA) {
        if (kAheadA > 0) {   // the next batch of the own row: into the L2, no register held
#pragma unroll
          for (int u = 0; u < kBatchA; ++u)
            if (i0 + kAheadA * kBatchA + u < cnt) prefetch_l2(z_img + s0 + (i0 + kAheadA * kBatchA + u) * NT);
        }
        uint4 rw[kBatchA];
#pragma unroll
        for (int u = 0; u < kBatchA; ++u)
          if (i0 + u < cnt) rw[u] = ldg_policy(z_img + s0 + (i0 + u) * NT, pol_keep);
        const float old = best;
#pragma unroll
        for (int u = 0; u < kBatchA; ++u) {
          if (i0 + u < cnt) {
            const float fm = SegOps<T>::to_float(SegOps<T>::fold(rw[u]));
            if (fm > best) { best = fm; best_seg = s0 + (i0 + u) * NT; }
          }
        }
        const float sc1 = EU::ex((old - best) * k1);
        s1p = __fmul2_rn(s1p, pair_of(sc1));
        s_1 *= sc1;
        const float2 nb1 = pair_of(-best * k1);
        float2 nbT = nb1;
        if (!t_one) {
          const float scT = EU::ex((old - best) * kT);
          sTp = __fmul2_rn(sTp, pair_of(scT));
          s_T *= scT;
          nbT = pair_of(-best * kT);
        }
#pragma unroll
        for (int u = 0; u < kBatchA; ++u) {
          if (i0 + u < cnt) {
            float2 z2[H];
            SegOps<T>::unpack2(rw[u], z2);
#pragma unroll
            for (int i = 0; i < H; ++i) {
              s1p = __fadd2_rn(s1p, ex_pair<T>(__ffma2_rn(z2[i], k1_2, nb1)));
              if (!t_one) sTp = __fadd2_rn(sTp, ex_pair<T>(__ffma2_rn(z2[i], kT_2, nbT)));
              zsp = __fadd2_rn(zsp, z2[i]);
            }
          }
        }
      }
      s_1 += s1p.x + s1p.y;
      s_T += sTp.x + sTp.y;
      z_sum += zsp.x + zsp.y;
    }
    if (edge) {
      float zv[V];
#pragma unroll
      for (int i = 0; i < V; ++i) {
        const int64_t c = (int64_t)edge_seg * V - g.head + i;
        zv[i] = (c >= 0 && c < C) ? Elem<T>::to_f32(z_row[c]) : -INFINITY;
      }
      own_values(zv, edge_seg);
    }
    float m, S = 0.f, S_T = 0.f, sum_z = 0.f;
    int m_seg;
    {
      const unsigned key = float_order_key(best + 0.f);  // -0 is folded onto +0: they tie
      const unsigned key_w = __reduce_max_sync(0xffffffffu, key);
      const int seg_w = (int)__reduce_min_sync(0xffffffffu, key == key_w ? (unsigned)best_seg : 0x7fffffffu);
      const float m_w = float_from_order_key(key_w);
      const float sw = warp_sum(s_1 * EU::ex((best - m_w) * k1));
      const float swT = warp_sum(s_T * EU::ex((best - m_w) * kT));
      const float zw = warp_sum(z_sum);
      if (lane == 0) { sh.red[par][warp] = make_float4(m_w, __int_as_float(seg_w), sw, zw); sh.red_t[par][warp] = swT; }
      __syncthreads();
      m = sh.red[par][0].x;
      m_seg = __float_as_int(sh.red[par][0].y);
#pragma unroll
      for (int wv = 1; wv < NW; ++wv) argmax_combine(m, m_seg, sh.red[par][wv].x, __float_as_int(sh.red[par][wv].y));
#pragma unroll
      for (int wv = 0; wv < NW; ++wv) {
        const float4 pt = sh.red[par][wv];
        S += pt.z * EU::ex((pt.x - m) * k1);
        S_T += sh.red_t[par][wv] * EU::ex((pt.x - m) * kT);
        sum_z += pt.w;
      }
      if (t_one) S_T = S;
    }
    if (m_seg >= g.n_seg) m_seg = 0;  // NaN rows: keep the reads below inside the row
    const int a_own = first_equal_global<T>(z_row, m_seg, g.head, C, m);
    const int seg_a = a.want_flags ? m_seg : -1;
    const float zy = Elem<T>::to_f32(z_row[y]);

    // ================= pass A2: softmax statistics of the peers (or of their mean) at temperature T
    float pm[NS], ps[NS];  // after the reduction: maximum and log_U of sum exp((x - max) / T)
    if (with_term) {
      float pb[NS], pa[NS];
#pragma unroll
      for (int q = 0; q < NS; ++q) { pb[q] = -3.0e38f; pa[q] = 0.f; }
      auto peer_values = [&](const float (&pv)[V], int q) {  // pv: values of one segment, -inf outside the row
        float fm = pv[0];
#pragma unroll
        for (int i = 1; i < V; ++i) fm = fmaxf(fm, pv[i]);
        const float old = pb[q];
        pb[q] = fmaxf(pb[q], fm);
        float acc = pa[q] * EU::ex((old - pb[q]) * kT);
#pragma unroll
        for (int i = 0; i < V; ++i)
          if (pv[i] != -INFINITY) acc += EU::ex((pv[i] - pb[q]) * kT);
        pa[q] = acc;
      };
      {
        // segments wholly inside the row: packed pairs; pa2[q] is relative to the running maximum pb[q]
        float2 pa2[NS];
#pragma unroll
        for (int q = 0; q < NS; ++q) pa2[q] = make_float2(0.f, 0.f);
        const float2 kT_2 = pair_of(kT), invP2 = pair_of(inv_P);
        auto peer_pairs = [&](const float2 (&x2)[H], int q) {
          float fm = fmaxf(x2[0].x, x2[0].y);
#pragma unroll
          for (int i = 1; i < H; ++i) fm = fmaxf(fm, fmaxf(x2[i].x, x2[i].y));
          const float old = pb[q];
          pb[q] = fmaxf(pb[q], fm);
          pa2[q] = __fmul2_rn(pa2[q], pair_of(EU::ex((old - pb[q]) * kT)));
          const float2 nb = pair_of(-pb[q] * kT);
#pragma unroll
          for (int i = 0; i < H; ++i) pa2[q] = __fadd2_rn(pa2[q], ex_pair<T>(__ffma2_rn(x2[i], kT_2, nb)));
        };
        for (int i0 = 0; i0 < cnt; ++i0) {
          const int s = s0 + i0 * NT;
          if (kAheadP > 0 && i0 + kAheadP < cnt) {   // the peers' segments a few iterations on
#pragma unroll
            for (int j = 0; j < P; ++j) prefetch_l2(p_img[j] + s + kAheadP * NT);
          }
          uint4 pr[PD];
#pragma unroll
          for (int j = 0; j < P; ++j) pr[j] = ldg_policy(p_img[j] + s, pol_keep);
          if constexpr (PW) {
#pragma unroll
            for (int j = 0; j < P; ++j) {
              float2 v2[H];
              SegOps<T>::unpack2(pr[j], v2);
              peer_pairs(v2, j);
            }
          } else {
            float2 zb2[H];
#pragma unroll
            for (int i = 0; i < H; ++i) zb2[i] = make_float2(0.f, 0.f);
#pragma unroll
            for (int j = 0; j < P; ++j) {
              float2 v2[H];
              SegOps<T>::unpack2(pr[j], v2);
#pragma unroll
              for (int i = 0; i < H; ++i) zb2[i] = __fadd2_rn(zb2[i], v2[i]);
            }
#pragma unroll
            for (int i = 0; i < H; ++i) zb2[i] = __fmul2_rn(zb2[i], invP2);
            peer_pairs(zb2, 0);
          }
        }
#pragma unroll
        for (int q = 0; q < NS; ++q) pa[q] = pa2[q].x + pa2[q].y;   // pa[q] was 0: the ragged segments come after
      }
      if (edge) {
        float zb[V];
#pragma unroll
        for (int i = 0; i < V; ++i) zb[i] = 0.f;
#pragma unroll
        for (int j = 0; j < P; ++j) {
          float pv[V];
#pragma unroll
          for (int i = 0; i < V; ++i) {
            const int64_t c = (int64_t)edge_seg * V - g.head + i;
            pv[i] = (c >= 0 && c < C) ? Elem<T>::to_f32(p_row[j][c]) : -INFINITY;
            zb[i] += pv[i];
          }
          if constexpr (PW) peer_values(pv, j);
        }
        if constexpr (!PW) {
#pragma unroll
          for (int i = 0; i < V; ++i) zb[i] *= inv_P;  // -inf stays -inf
          peer_values(zb, 0);
        }
      }
#pragma unroll
      for (int q = 0; q < NS; ++q) {
        const float mw = warp_max_redux(pb[q]);
        const float sw = warp_sum(pa[q] * EU::ex((pb[q] - mw) * kT));
        if (lane == 0) sh.peer[par][q][warp] = make_float2(mw, sw);
      }
      __syncthreads();
#pragma unroll
      for (int q = 0; q < NS; ++q) {
        float mq = sh.peer[par][q][0].x;
#pragma unroll
        for (int wv = 1; wv < NW; ++wv) mq = fmaxf(mq, sh.peer[par][q][wv].x);
        float sq = 0.f;
#pragma unroll
        for (int wv = 0; wv < NW; ++wv) sq += sh.peer[par][q][wv].y * EU::ex((sh.peer[par][q][wv].x - mq) * kT);
        pm[q] = mq;
        ps[q] = EU::lg(sq);
      }
    } else {
#pragma unroll
      for (int q = 0; q < NS; ++q) { pm[q] = 0.f; ps[q] = 0.f; }
    }

    // ================= pass B: distance and gradient
    // exponent arguments in U: own at T = 1: z k1 - c1; own at T: z kT - cT; peer statistic q: x kT - cq[q]
    const float c1 = m * k1, cT = m * kT + EU::lg(S_T);
    float cq[NS];
#pragma unroll
    for (int q = 0; q < NS; ++q) cq[q] = pm[q] * kT + ps[q];
    const float cp = w * __frcp_rn(S);                      // exp(z - m) -> w p
    const float cq_smooth = w * a.eps * inv_C;
    const float cy = w * (1.f - a.eps);
    const float cg = with_term ? w * a.alpha * temp : 0.f;  // (p^T - tbar) -> w alpha dD/dz
    const float t_scale = PW ? inv_P : 1.f;                 // tbar = t_scale * sum of the t's
    float dacc = 0.f;                                        // sum t (log_U t - log_U p^T)
    float lt[PD], ge[PD], za[PD];
#pragma unroll
    for (int j = 0; j < PD; ++j) { lt[j] = -INFINITY; ge[j] = -INFINITY; za[j] = -INFINITY; }
    // one column: own value z, peer values pv[]; returns the gradient element
    auto column = [&](float z, const float (&pv)[PD], int64_t c) -> float {
      const float e = EU::ex(fmaf(z, k1, -c1));
      const float lpT = fmaf(z, kT, -cT);
      float gv = fmaf(e, cp, -cq_smooth);
      if (c == (int64_t)y) gv -= cy;
      if (with_term) {
        const float pT = EU::ex(lpT);
        float tsum = 0.f;
        if constexpr (PW) {
#pragma unroll
          for (int j = 0; j < P; ++j) {
            const float l = fmaf(pv[j], kT, -cq[j]);
            const float t = EU::ex(l);
            tsum += t;
            dacc = fmaf(t, l - lpT, dacc);
          }
        } else {
          float zb = 0.f;
#pragma unroll
          for (int j = 0; j < P; ++j) zb += pv[j];
          const float l = fmaf(zb * inv_P, kT, -cq[0]);
          const float t = EU::ex(l);
          tsum = t;
          dacc = fmaf(t, l - lpT, dacc);
        }
        gv = fmaf(cg, pT - tsum * t_scale, gv);
      }
      if (a.want_flags) {
#pragma unroll
        for (int j = 0; j < P; ++j) {
          if (c < a_own) lt[j] = fmaxf(lt[j], pv[j]);
          else if (c > a_own) ge[j] = fmaxf(ge[j], pv[j]);
          else za[j] = pv[j];
        }
      }
      return gv;
    };
    // segments wholly inside the row: packed pairs
    typename SegOps<T>::macc ltp[PD], gep[PD];
#pragma unroll
    for (int j = 0; j < PD; ++j) { ltp[j] = SegOps<T>::neg_inf(); gep[j] = SegOps<T>::neg_inf(); }
    {
      const float2 k1_2 = pair_of(k1), nc1_2 = pair_of(-c1), kT_2 = pair_of(kT), ncT_2 = pair_of(-cT);
      const float2 cp2 = pair_of(cp), ncq2 = pair_of(-cq_smooth), cg2 = pair_of(cg), nts2 = pair_of(-t_scale);
      const float2 invS2 = pair_of(__frcp_rn(S)), invP2 = pair_of(inv_P), neg1 = pair_of(-1.f);
      const int seg_y = (g.head + y) / V, pos_y = (g.head + y) % V;
      float2 dacc2 = make_float2(0.f, 0.f);
      for (int i0 = 0; i0 < cnt; ++i0) {
        const int s = s0 + i0 * NT;
        const uint4 zr = z_img[s];
        uint4 pr[PD];
        if (stream_peers) {
#pragma unroll
          for (int j = 0; j < P; ++j) pr[j] = p_img[j][s];
        }
        float2 z2[H], g2[H], lp2[H], pT2[H];
        SegOps<T>::unpack2(zr, z2);
#pragma unroll
        for (int i = 0; i < H; ++i) {
          const float2 e = ex_pair<T>(__ffma2_rn(z2[i], k1_2, nc1_2));
          lp2[i] = __ffma2_rn(z2[i], kT_2, ncT_2);
          g2[i] = __ffma2_rn(e, cp2, ncq2);
          pT2[i] = e;
          if (with_term) pT2[i] = t_one ? __fmul2_rn(e, invS2) : ex_pair<T>(lp2[i]);
        }
        if (with_term) {
          float2 ts2[H];
#pragma unroll
          for (int i = 0; i < H; ++i) ts2[i] = make_float2(0.f, 0.f);
          if constexpr (PW) {
#pragma unroll
            for (int j = 0; j < P; ++j) {
              float2 v2[H];
              SegOps<T>::unpack2(pr[j], v2);
              const float2 ncq_j = pair_of(-cq[j]);
#pragma unroll
              for (int i = 0; i < H; ++i) {
                const float2 l = __ffma2_rn(v2[i], kT_2, ncq_j);
                const float2 t = ex_pair<T>(l);
                ts2[i] = __fadd2_rn(ts2[i], t);
                dacc2 = __ffma2_rn(t, __ffma2_rn(lp2[i], neg1, l), dacc2);
              }
            }
          } else {
            float2 zb2[H];
#pragma unroll
            for (int i = 0; i < H; ++i) zb2[i] = make_float2(0.f, 0.f);
#pragma unroll
            for (int j = 0; j < P; ++j) {
              float2 v2[H];
              SegOps<T>::unpack2(pr[j], v2);
#pragma unroll
              for (int i = 0; i < H; ++i) zb2[i] = __fadd2_rn(zb2[i], v2[i]);
            }
            const float2 ncq_0 = pair_of(-cq[0]);
#pragma unroll
            for (int i = 0; i < H; ++i) {
              const float2 l = __ffma2_rn(__fmul2_rn(zb2[i], invP2), kT_2, ncq_0);
              const float2 t = ex_pair<T>(l);
              ts2[i] = t;
              dacc2 = __ffma2_rn(t, __ffma2_rn(lp2[i], neg1, l), dacc2);
            }
          }
#pragma unroll
          for (int i = 0; i < H; ++i) g2[i] = __ffma2_rn(__ffma2_rn(ts2[i], nts2, pT2[i]), cg2, g2[i]);
        }
        if (a.want_flags) {
#pragma unroll
          for (int j = 0; j < P; ++j) {
            const typename SegOps<T>::macc f = SegOps<T>::fold(pr[j]);
            const bool before = s < seg_a;
            ltp[j] = before ? SegOps<T>::mmax(ltp[j], f) : ltp[j];
            gep[j] = before ? gep[j] : SegOps<T>::mmax(gep[j], f);
            if (s == seg_a) {
              // The segment of the own arg-max column a went to ge as a whole.  The peer's value at a and the
              // largest value before a inside the segment settle the rest (see rows_stream.cu).
              float vv[V];
              SegOps<T>::unpack(pr[j], vv);
              float pre = -INFINITY;
#pragma unroll
              for (int i = 0; i < V; ++i) {
                const int c = seg_a * V - g.head + i;
                if (c < a_own) pre = fmaxf(pre, vv[i]);
                if (c == a_own) za[j] = vv[i];
              }
              lt[j] = fmaxf(lt[j], pre);
            }
          }
        }
        if (s == seg_y) {  // the label column: q_y carries the extra 1 - eps
#pragma unroll
          for (int i = 0; i < H; ++i) {
            if (2 * i == pos_y) g2[i].x -= cy;
            if (2 * i + 1 == pos_y) g2[i].y -= cy;
          }
        }
        if (g_img) g_img[s] = SegOps<T>::pack2(g2);
      }
      dacc += dacc2.x + dacc2.y;
    }
    if (edge) {
#pragma unroll
      for (int i = 0; i < V; ++i) {
        const int64_t c = (int64_t)edge_seg * V - g.head + i;
        if (c < 0 || c >= C) continue;
        float pv[PD];
#pragma unroll
        for (int j = 0; j < PD; ++j) pv[j] = (stream_peers && j < P) ? Elem<T>::to_f32(p_row[j][c]) : 0.f;
        const float gvv = column(Elem<T>::to_f32(z_row[c]), pv, c);
        if (g_row) g_row[c] = Elem<T>::from_f32(gvv);
      }
    }

    // ================= row results: per-warp partials, then warp 0 finishes the row
    {
      float part[1 + 3 * PD];
      part[0] = warp_sum(dacc);
#pragma unroll
      for (int j = 0; j < PD; ++j) {
        part[1 + 3 * j] = warp_max_redux(fmaxf(lt[j], SegOps<T>::to_float(ltp[j])));
        part[2 + 3 * j] = warp_max_redux(fmaxf(ge[j], SegOps<T>::to_float(gep[j])));
        part[3 + 3 * j] = warp_max_redux(za[j]);
      }
      if (lane == 0) {
#pragma unroll
        for (int i = 0; i < 1 + 3 * PD; ++i) sh.endred[par][i * NW + warp] = part[i];
      }
      __syncthreads();
      if (warp == 0) {
        const float* er = sh.endred[par];
        const float dsum = warp_sum(lane < NW ? er[lane] : 0.f);
        uint32_t flags = 0u;
        if (a.want_flags) {
          flags = (a_own == y) ? 1u : 0u;
#pragma unroll
          for (int j = 0; j < P; ++j) {
            const float ltv = warp_max_redux(lane < NW ? er[(1 + 3 * j) * NW + lane] : -INFINITY);
            const float gev = warp_max_redux(lane < NW ? er[(2 + 3 * j) * NW + lane] : -INFINITY);
            const float zav = warp_max_redux(lane < NW ? er[(3 + 3 * j) * NW + lane] : -INFINITY);
            if (zav >= gev && ltv < zav) flags |= (2u << j);
          }
        }
        if (lane == 0) {
          const float ce = (m + logf(S)) - (1.f - a.eps) * zy - (a.eps * inv_C) * sum_z;
          float D = 0.f;
          if (with_term) D = temp * temp * (dsum / EU::kU) * t_scale;
          a.row_loss[r] = with_term ? fmaf(a.alpha, D, ce) : ce;
          a.row_flags[r] = flags;
        }
      }
    }
    ++v;
  }

  // ---------------- all rows of this CTA are written: scheduler reset and final reduction
  if (stream_last_cta(a.hdr, &sh.last_flag, tid) && a.fused_finalize) {
    __threadfence();
    finalize_cta(a, sh.fin);
  }
}

// ------------------------------------------------------------------ host side
template <typename T, int P, bool PW>
static cudaError_t stream_kl_launch_one(const KArgs& a, int grid, cudaStream_t stream) {
  const cudaError_t e = launch_overlapped(rows_stream_kl_kernel<T, P, PW>, dim3(grid), dim3(stream_threads(P)), 0, stream, a);
  return e != cudaSuccess ? e : cudaGetLastError();
}

template <typename T>
static cudaError_t stream_kl_launch_peers(const KArgs& a, int grid, cudaStream_t stream) {
  const bool pw = a.peer_reduce == CODISTILL_PEERS_PAIRWISE_MEAN;
  switch (a.n_peers) {
    case 0: return stream_kl_launch_one<T, 0, true>(a, grid, stream);
    case 1: return pw ? stream_kl_launch_one<T, 1, true>(a, grid, stream) : stream_kl_launch_one<T, 1, false>(a, grid, stream);
    case 2: return pw ? stream_kl_launch_one<T, 2, true>(a, grid, stream) : stream_kl_launch_one<T, 2, false>(a, grid, stream);
    case 3: return pw ? stream_kl_launch_one<T, 3, true>(a, grid, stream) : stream_kl_launch_one<T, 3, false>(a, grid, stream);
    case 7: return pw ? stream_kl_launch_one<T, 7, true>(a, grid, stream) : stream_kl_launch_one<T, 7, false>(a, grid, stream);
    default: return cudaErrorNotSupported;
  }
}

cudaError_t launch_stream_kl(const KArgs& a, int dtype, int num_sms, cudaStream_t stream) {
  const int64_t rows = a.row_end - a.row_begin;
  if (rows <= 0) return cudaSuccess;
  const int64_t slots = (int64_t)num_sms * stream_kl_ctas_per_sm(a.n_peers);
  const int grid = (int)(rows < slots ? rows : slots);
  return dtype == CODISTILL_F32 ? stream_kl_launch_peers<float>(a, grid, stream) : stream_kl_launch_peers<__nv_bfloat16>(a, grid, stream);
}

}  // namespace codistill
