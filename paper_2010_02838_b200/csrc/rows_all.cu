// All n models in one call (Algorithm 1's inner loop over the models i = 1..n, on one minibatch):
// every model's objective with the other n-1 models as its peers, MSE-on-logits distance.
//
// (With the centred distance every model's logits first lose their mean over the classes, known after pass A.)
// Per column c the n logits z_1..z_n of a row are centred on their mean mu_c, z'_i = z_i - mu_c.  Then
//   z_i - zbar_(-i)            = n / (n-1) * z'_i                        (zbar_(-i): mean of the other models)
//   sum_{j != i} (z_i - z_j)^2 = n * z'_i^2 + sum_j z'_j^2               (no cancellation: all terms >= 0)
// so the distance and its gradient of all n models come from one read of the n rows, instead of n
// reads of each row by n separate calls.  Organisation as in rows_stream.cu: one CTA per row index,
// nothing staged, 16-byte loads;
//   pass A  the n rows: per model the online softmax statistics and the first arg-max;
//   pass B  the n rows again: centring, distance terms, the n gradient rows.
// Arg-max agreement between models i and j is a_i == a_j: all arg-maxes are known after pass A.
//
// KL distance (pairwise over the peers): with t_j = softmax(z_j / T), Q_c = sum_j t_jc and
// E_c = sum_j t_jc log t_jc,
//   sum_{j != i} KL(t_j || t_i)          = sum_c (E_c - Q_c log t_ic)
//   d/dz_ic of T^2 sum_{j != i} KL(..)   = T (n t_ic - Q_c)
// so again one read of the n rows per pass serves all n models; pass A adds sum_c exp((z - m) / T).
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <type_traits>

#include "cluster_args.cuh"
#include "stream_common.cuh"

namespace codistill {

constexpr int kAllMax = CODISTILL_ALL_MAX_MODELS;
__host__ __device__ constexpr int all_threads(int n) { return n >= 5 ? 128 : 256; }
// CTAs per SM.  Five and more models run 128-thread CTAs: four per SM for the KL form, three for the MSE forms (168
// registers per thread and next to no spills instead of 128 with spills: workload 5, all 8 models, 6.94 -> 6.45 ms;
// the KL form was 10 % slower that way, and two CTAs per SM were slower for both).
__host__ __device__ constexpr int all_ctas_per_sm(int n, bool kl) { return n >= 5 ? (kl ? 4 : 3) : 3; }

struct AllArgs {
  const void* model[kAllMax];
  void* grad[kAllMax];          // all set or all null (forward only)
  const int32_t* labels;
  const uint8_t* mask;          // nullable
  float* row_loss;              // [n][rows]
  uint32_t* row_flags;          // [n][rows]
  WsHeader* hdr;
  const int64_t* partials;
  float* reduced_loss;          // [n]
  int64_t* counters;            // [n][3 + (n-1)], nullable
  int32_t* dev_status;          // nullable
  int64_t rows, classes, row_stride;
  int n, peer_reduce, reduction;
  int centred;                  // distance between logits centred on their class means
  float alpha, eps;
  float temperature;            // KL distance only
};

struct AllRowStat { float m, S, sum_z, zy; int a_own; };

struct AllShared {
  float4 red[2][kAllMax][kStreamMaxWarps];   // pass A partials per model: max, first segment, sum exp, sum z
  float dist[2][kAllMax][kStreamMaxWarps];   // pass B partials per model
  float red_t[2][kAllMax][kStreamMaxWarps];  // KL: sum exp((z - m) / T) partials per model
  AllRowStat stat[2][kAllMax];
  long long next_row[2];
  double fin[32];
  int last_flag;
};

// the columns of one 32-bit word of a segment
template <typename T> struct WordOps;
template <> struct WordOps<float> {
  static constexpr int G = 1;
  __device__ static void unpack(uint32_t w, float (&o)[1]) { o[0] = __uint_as_float(w); }
  __device__ static uint32_t pack(const float (&g)[1]) { return __float_as_uint(g[0]); }
};
template <> struct WordOps<__nv_bfloat16> {
  static constexpr int G = 2;
  __device__ static void unpack(uint32_t w, float (&o)[2]) { o[0] = __uint_as_float(w << 16); o[1] = __uint_as_float(w & 0xFFFF0000u); }
  __device__ static uint32_t pack(const float (&g)[2]) {
    const __nv_bfloat162 p = __floats2bfloat162_rn(g[0], g[1]);
    return *reinterpret_cast<const uint32_t*>(&p);
  }
};

// Iterations a thread's segments are requested ahead of their loads.  The MSE forms wait on memory most of
// the time and gain 6-15 %; the KL form is bound by arithmetic and the extra instructions cost it 3 %.
__host__ __device__ constexpr int all_ahead(int n, bool kl) { return kl ? 0 : n >= 5 ? 1 : 2; }

// exp(x), x in natural units: full precision for fp32 logits, the hardware exp2 for bf16 logits
template <typename T>
__device__ __forceinline__ float exp_nat(float x) {
  if constexpr (sizeof(T) == 4) return expf(x); else return ex2_approx(x * kLog2e);
}

template <typename T, int N, bool PW, bool KL>
__global__ void __launch_bounds__(all_threads(N), all_ctas_per_sm(N, KL)) rows_all_kernel(const __grid_constant__ AllArgs a) {
  constexpr int V = SegOps<T>::V;
  constexpr int G = WordOps<T>::G;
  constexpr int NT = all_threads(N);
  constexpr int NW = NT / 32;
  constexpr int kAhead = all_ahead(N, KL);
  __shared__ AllShared sh;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t C = a.classes, R = a.rows;
  const bool with_term = a.alpha != 0.f;

  wait_for_prior_grid();  // from here on the workspace header and the valid-row counts are read
  float w = 1.f;
  if (a.reduction == CODISTILL_REDUCE_MEAN_VALID) {
    const int nb = a.hdr->prep_blocks;
    int64_t nv = 0;
    for (int b = 0; b < nb; ++b) nv += a.partials[2 * b];
    w = 1.f / (float)(nv > 1 ? nv : 1);
  }
  const float inv_C = 1.f / (float)C;
  const bool need_z = a.eps != 0.f || a.centred != 0;
  constexpr float kRatio = (float)N / (float)(N - 1);           // z_i - zbar_(-i) = kRatio * z'_i
  const float cd = with_term ? w * a.alpha * (2.f * inv_C) * kRatio : 0.f;  // z'_i -> w alpha dD_i/dz_i
  const float cq = w * a.eps * inv_C;
  const float cy = w * (1.f - a.eps);
  const float inv_T = KL ? 1.f / a.temperature : 1.f;
  const bool t_one = a.temperature == 1.f;
  const float ckl = with_term ? w * a.alpha * a.temperature / (float)(N - 1) : 0.f;  // (n t_i - Q) -> w alpha dD_i/dz_i

  stream_draw_row(&sh.next_row[0], a.hdr, 0, tid);
  __syncthreads();
  int v = 0;  // valid rows done by this CTA
  for (int it = 0;; ++it) {
    const long long r = sh.next_row[it & 1];
    if (r >= R) break;
    stream_draw_row(&sh.next_row[(it + 1) & 1], a.hdr, 0, tid);
    const StreamRow row = stream_row<T, NT>(r, r, a.row_stride, C, a.labels, a.mask, tid);
    const RowGeom g = row.g;
    const int64_t row_off = row.row_off;  // in elements
    const int cnt = row.cnt, s0 = row.s0, y = row.y, edge_seg = row.edge_seg;
    const bool edge = row.edge;
    const T* z_row[N];
    const uint4* z_img[N];
#pragma unroll
    for (int i = 0; i < N; ++i) {
      z_row[i] = reinterpret_cast<const T*>(a.model[i]) + row_off;
      z_img[i] = reinterpret_cast<const uint4*>(z_row[i] - g.head);
    }
    const bool want_grad = a.grad[0] != nullptr;

    if (!row.valid) {  // masked row: zero gradient rows, no loss, no counts; nothing is read
      if (want_grad) {
#pragma unroll
        for (int i = 0; i < N; ++i) stream_zero_row<T, NT>(reinterpret_cast<T*>(a.grad[i]) + row_off, row, C);
      }
      if (tid < N) { a.row_loss[(int64_t)tid * R + r] = 0.f; a.row_flags[(int64_t)tid * R + r] = 0u; }
      __syncthreads();  // orders the row-id hand-over
      continue;
    }
    const int par = v & 1;

    // ================= pass A: per model, online softmax statistics and first arg-max segment
    float best[N], s_acc[N], z_acc[N], t_acc[N];
    int best_seg[N];
#pragma unroll
    for (int i = 0; i < N; ++i) { best[i] = -3.0e38f; best_seg[i] = 0x7fffffff; s_acc[i] = 0.f; z_acc[i] = 0.f; t_acc[i] = 0.f; }
    auto stats_values = [&](const float (&zv)[V], int s, float& bst, int& bsg, float& sa, float& za, float& ta) {
      float fm = zv[0];
#pragma unroll
      for (int e = 1; e < V; ++e) fm = fmaxf(fm, zv[e]);
      const float old = bst;
      if (fm > bst || (fm == bst && s < bsg)) { bst = fm; bsg = s; }
      float acc = sa * rescale_exp2<T>((old - bst) * kLog2e);
      const float nm = -bst * kLog2e;
#pragma unroll
      for (int e = 0; e < V; ++e) {
        if (zv[e] != -INFINITY) {
          acc += exp_shift2<T>(make_float2(zv[e], zv[e]), bst, make_float2(kLog2e, kLog2e), make_float2(nm, nm)).x;
          za += zv[e];
        }
      }
      sa = acc;
      if constexpr (KL) {
        if (!t_one) {
          float acc_t = ta * exp_nat<T>((old - bst) * inv_T);
#pragma unroll
          for (int e = 0; e < V; ++e) acc_t += exp_nat<T>((zv[e] - bst) * inv_T);   // exp(-inf) = 0: columns outside the row
          ta = acc_t;
        }
      }
    };
    // whole segments: packed pairs (a thread meets its segments in increasing order, so a strictly larger
    // maximum is the first one); the tempered sum of the KL form at T != 1 takes the element-wise path
    const bool packed_a = !KL || t_one;
    if (packed_a) {
      constexpr int H = SegOps<T>::H;
      float2 s2[N], zs2[N];
#pragma unroll
      for (int i = 0; i < N; ++i) { s2[i] = make_float2(0.f, 0.f); zs2[i] = make_float2(0.f, 0.f); }
      for (int k = 0; k < cnt; ++k) {
        const int s = s0 + k * NT;
        if (kAhead > 0 && k + kAhead < cnt) {
#pragma unroll
          for (int i = 0; i < N; ++i) prefetch_l2(z_img[i] + s + kAhead * NT);
        }
        uint4 rw[N];
#pragma unroll
        for (int i = 0; i < N; ++i) rw[i] = z_img[i][s];
#pragma unroll
        for (int i = 0; i < N; ++i) {
          const float fm = SegOps<T>::to_float(SegOps<T>::fold(rw[i]));
          const float old = best[i];
          if (fm > best[i]) { best[i] = fm; best_seg[i] = s; }
          const float sc = rescale_exp2<T>((old - best[i]) * kLog2e);
          const float nm = -best[i] * kLog2e;
          float2 acc = __fmul2_rn(s2[i], make_float2(sc, sc));
          float2 z2[H];
          SegOps<T>::unpack2(rw[i], z2);
#pragma unroll
          for (int h = 0; h < H; ++h) acc = __fadd2_rn(acc, exp_shift2<T>(z2[h], best[i], make_float2(kLog2e, kLog2e), make_float2(nm, nm)));
          if (need_z) {   // the sum of the logits: label smoothing and the centred distance only
#pragma unroll
            for (int h = 0; h < H; ++h) zs2[i] = __fadd2_rn(zs2[i], z2[h]);
          }
          s2[i] = acc;
        }
      }
#pragma unroll
      for (int i = 0; i < N; ++i) { s_acc[i] = s2[i].x + s2[i].y; z_acc[i] = zs2[i].x + zs2[i].y; }
    } else {
      for (int k = 0; k < cnt; ++k) {
        const int s = s0 + k * NT;
        uint4 rw[N];
#pragma unroll
        for (int i = 0; i < N; ++i) rw[i] = z_img[i][s];
#pragma unroll
        for (int i = 0; i < N; ++i) {
          float zv[V];
          SegOps<T>::unpack(rw[i], zv);
          stats_values(zv, s, best[i], best_seg[i], s_acc[i], z_acc[i], t_acc[i]);
        }
      }
    }
    if (edge) {
#pragma unroll
      for (int i = 0; i < N; ++i) {
        float zv[V];
#pragma unroll
        for (int e = 0; e < V; ++e) {
          const int64_t c = (int64_t)edge_seg * V - g.head + e;
          zv[e] = (c >= 0 && c < C) ? Elem<T>::to_f32(z_row[i][c]) : -INFINITY;
        }
        stats_values(zv, edge_seg, best[i], best_seg[i], s_acc[i], z_acc[i], t_acc[i]);
      }
    }
#pragma unroll
    for (int i = 0; i < N; ++i) {
      const unsigned key = float_order_key(best[i] + 0.f);  // -0 is folded onto +0: they tie
      const unsigned key_w = __reduce_max_sync(0xffffffffu, key);
      const int seg_w = (int)__reduce_min_sync(0xffffffffu, key == key_w ? (unsigned)best_seg[i] : 0x7fffffffu);
      const float m_w = float_from_order_key(key_w);
      const float sw = warp_sum(s_acc[i] * rescale_exp2<T>((best[i] - m_w) * kLog2e));
      const float zw = warp_sum(z_acc[i]);
      if (lane == 0) sh.red[par][i][warp] = make_float4(m_w, __int_as_float(seg_w), sw, zw);
      if constexpr (KL) {
        const float tw = warp_sum(t_acc[i] * exp_nat<T>((best[i] - m_w) * inv_T));
        if (lane == 0) sh.red_t[par][i][warp] = tw;
      }
    }
    __syncthreads();
    float mi[N], cpi[N], cmi[N];  // per model: maximum, w / S, class mean removed before the distance (0: plain MSE)
    float cti[KL ? N : 1], lsi[KL ? N : 1];  // KL: 1 / S_T and log S_T, S_T = sum_c exp((z_c - m) / T)
    int a_own[N];
#pragma unroll
    for (int i = 0; i < N; ++i) {
      float m = sh.red[par][i][0].x;
      int m_seg = __float_as_int(sh.red[par][i][0].y);
#pragma unroll
      for (int wv = 1; wv < NW; ++wv) argmax_combine(m, m_seg, sh.red[par][i][wv].x, __float_as_int(sh.red[par][i][wv].y));
      float S = 0.f, sum_z = 0.f;
#pragma unroll
      for (int wv = 0; wv < NW; ++wv) {
        const float4 pt = sh.red[par][i][wv];
        S += pt.z * rescale_exp2<T>((pt.x - m) * kLog2e);
        sum_z += pt.w;
      }
      if (m_seg >= g.n_seg) m_seg = 0;  // NaN rows: keep the reads below inside the row
      a_own[i] = first_equal_global<T>(z_row[i], m_seg, g.head, C, m);
      mi[i] = m;
      cpi[i] = w * __frcp_rn(S);
      cmi[i] = sum_z * inv_C;   // class mean; turned into (average class mean) - (class mean) below
      if constexpr (KL) {
        float S_T = S;
        if (!t_one) {
          S_T = 0.f;
#pragma unroll
          for (int wv = 0; wv < NW; ++wv) S_T += sh.red_t[par][i][wv] * exp_nat<T>((sh.red[par][i][wv].x - m) * inv_T);
        }
        cti[i] = __frcp_rn(S_T);
        lsi[i] = logf(S_T);
      }
      if (tid == 0) {
        AllRowStat st;
        st.m = m; st.S = S; st.sum_z = sum_z; st.zy = Elem<T>::to_f32(z_row[i][y]); st.a_own = a_own[i];
        sh.stat[par][i] = st;
      }
    }

    {
      float avg = 0.f;
#pragma unroll
      for (int i = 0; i < N; ++i) avg += cmi[i];
      avg *= (1.f / (float)N);
#pragma unroll
      for (int i = 0; i < N; ++i) cmi[i] = avg - cmi[i];
    }

    // ================= pass B: centring, distance terms, gradients
    float dist[N];
#pragma unroll
    for (int i = 0; i < N; ++i) dist[i] = 0.f;
    // one column: values zc[] of the n models; returns the gradient elements in gc[]
    auto column = [&](const float (&zc)[N], float (&gc)[N], int64_t c) {
      if constexpr (KL) {
        const float cqc = (c == (int64_t)y) ? cq + cy : cq;
        float t[N], lt[N], Q = 0.f, E = 0.f;
#pragma unroll
        for (int i = 0; i < N; ++i) {
          const float x = zc[i] - mi[i];
          const float e1 = exp_nat<T>(x);
          t[i] = (t_one ? e1 : exp_nat<T>(x * inv_T)) * cti[i];
          lt[i] = fmaxf(fmaf(x, inv_T, -lsi[i]), -3.0e38f);   // log t_i, kept finite so that 0 * log 0 = 0
          Q += t[i];
          E = fmaf(t[i], lt[i], E);
          gc[i] = fmaf(e1, cpi[i], -cqc);
        }
#pragma unroll
        for (int i = 0; i < N; ++i) {
          gc[i] = fmaf(ckl, fmaf((float)N, t[i], -Q), gc[i]);
          dist[i] += fmaf(-Q, lt[i], E);                       // sum_{j != i} t_j (log t_j - log t_i)
        }
        return;
      }
      // z'_i = z_i - mean_j z_j; the centred distance adds cmi[i] = (average class mean) - (class mean of model i)
      float zp[N], mu = zc[0];
#pragma unroll
      for (int i = 1; i < N; ++i) mu += zc[i];
      mu *= (-1.f / (float)N);
#pragma unroll
      for (int i = 0; i < N; ++i) zp[i] = zc[i] + mu;
      if (a.centred) {
#pragma unroll
        for (int i = 0; i < N; ++i) zp[i] += cmi[i];
      }
      const float cqc = (c == (int64_t)y) ? cq + cy : cq;
#pragma unroll
      for (int i = 0; i < N; ++i) {
        const float e = exp_shift2<T>(make_float2(zc[i], zc[i]), mi[i], make_float2(kLog2e, kLog2e),
                                      make_float2(-mi[i] * kLog2e, -mi[i] * kLog2e)).x;
        gc[i] = fmaf(e, cpi[i], fmaf(cd, zp[i], -cqc));
        dist[i] = fmaf(zp[i], zp[i], dist[i]);   // z'_i^2 = (z_i - zbar_(-i))^2 / kRatio^2; pairwise form: see the row results
      }
    };
    [[maybe_unused]] float2 dist2[N];
#pragma unroll
    for (int i = 0; i < N; ++i) dist2[i] = make_float2(0.f, 0.f);
    // two neighbouring columns c, c + 1 of the n models at once (packed fp32 pairs; bf16 logits)
    auto column2 = [&](const float2 (&zc)[N], float2 (&gc)[N], int64_t c) {
      if constexpr (KL) {
        const float2 ncq = make_float2((c == (int64_t)y) ? -(cq + cy) : -cq, (c + 1 == (int64_t)y) ? -(cq + cy) : -cq);
        const float2 l2e = make_float2(kLog2e, kLog2e), l2e_T = make_float2(kLog2e * inv_T, kLog2e * inv_T);
        float2 t[N], lt[N], Q = make_float2(0.f, 0.f), E = make_float2(0.f, 0.f);
#pragma unroll
        for (int i = 0; i < N; ++i) {
          const float2 x = __fadd2_rn(zc[i], make_float2(-mi[i], -mi[i]));
          const float2 a1 = __fmul2_rn(x, l2e);
          const float2 e1 = make_float2(ex2_approx(a1.x), ex2_approx(a1.y));
          float2 et = e1;
          if (!t_one) {
            const float2 aT = __fmul2_rn(x, l2e_T);
            et = make_float2(ex2_approx(aT.x), ex2_approx(aT.y));
          }
          t[i] = __fmul2_rn(et, make_float2(cti[i], cti[i]));
          const float2 l = __ffma2_rn(x, make_float2(inv_T, inv_T), make_float2(-lsi[i], -lsi[i]));
          lt[i] = make_float2(fmaxf(l.x, -3.0e38f), fmaxf(l.y, -3.0e38f));   // log t_i, kept finite: 0 * log 0 = 0
          Q = __fadd2_rn(Q, t[i]);
          E = __ffma2_rn(t[i], lt[i], E);
          gc[i] = __ffma2_rn(e1, make_float2(cpi[i], cpi[i]), ncq);
        }
        const float2 nQ = make_float2(-Q.x, -Q.y);
#pragma unroll
        for (int i = 0; i < N; ++i) {
          gc[i] = __ffma2_rn(make_float2(ckl, ckl), __ffma2_rn(make_float2((float)N, (float)N), t[i], nQ), gc[i]);
          dist2[i] = __fadd2_rn(dist2[i], __ffma2_rn(nQ, lt[i], E));   // sum_{j != i} t_j (log t_j - log t_i)
        }
        return;
      }
      float2 zp[N], mu = zc[0];
#pragma unroll
      for (int i = 1; i < N; ++i) mu = __fadd2_rn(mu, zc[i]);
      mu = __fmul2_rn(mu, make_float2(-1.f / (float)N, -1.f / (float)N));
#pragma unroll
      for (int i = 0; i < N; ++i) zp[i] = __fadd2_rn(zc[i], mu);
      if (a.centred) {
#pragma unroll
        for (int i = 0; i < N; ++i) zp[i] = __fadd2_rn(zp[i], make_float2(cmi[i], cmi[i]));
      }
      const float2 ncq = make_float2((c == (int64_t)y) ? -(cq + cy) : -cq, (c + 1 == (int64_t)y) ? -(cq + cy) : -cq);
#pragma unroll
      for (int i = 0; i < N; ++i) {
        const float nm = -mi[i] * kLog2e;
        const float2 e = exp_shift2<T>(zc[i], mi[i], make_float2(kLog2e, kLog2e), make_float2(nm, nm));
        gc[i] = __ffma2_rn(e, make_float2(cpi[i], cpi[i]), __ffma2_rn(make_float2(cd, cd), zp[i], ncq));
        dist2[i] = __ffma2_rn(zp[i], zp[i], dist2[i]);
      }
    };
    constexpr bool kPackedB = (G == 2);
    if constexpr (kPackedB) {
      for (int k = 0; k < cnt; ++k) {
        const int s = s0 + k * NT;
        if (kAhead > 0 && k + kAhead < cnt) {
#pragma unroll
          for (int i = 0; i < N; ++i) prefetch_l2(z_img[i] + s + kAhead * NT);
        }
        uint4 rw[N];
#pragma unroll
        for (int i = 0; i < N; ++i) rw[i] = z_img[i][s];
        const int64_t cbase = (int64_t)s * V - g.head;
#pragma unroll
        for (int wd = 0; wd < 4; ++wd) {
          float2 zc[N], gc[N];
#pragma unroll
          for (int i = 0; i < N; ++i) {
            const uint32_t word = wd == 0 ? rw[i].x : wd == 1 ? rw[i].y : wd == 2 ? rw[i].z : rw[i].w;
            zc[i] = make_float2(__uint_as_float(word << 16), __uint_as_float(word & 0xFFFF0000u));
          }
          column2(zc, gc, cbase + wd * 2);
#pragma unroll
          for (int i = 0; i < N; ++i) {
            const __nv_bfloat162 pk = __floats2bfloat162_rn(gc[i].x, gc[i].y);
            const uint32_t word = *reinterpret_cast<const uint32_t*>(&pk);
            if (wd == 0) rw[i].x = word; else if (wd == 1) rw[i].y = word; else if (wd == 2) rw[i].z = word; else rw[i].w = word;
          }
        }
        if (want_grad) {
#pragma unroll
          for (int i = 0; i < N; ++i)
            reinterpret_cast<uint4*>(reinterpret_cast<T*>(a.grad[i]) + row_off - g.head)[s] = rw[i];
        }
      }
    }
    for (int k = 0; k < (kPackedB ? 0 : cnt); ++k) {
      const int s = s0 + k * NT;
      uint4 rw[N];
#pragma unroll
      for (int i = 0; i < N; ++i) rw[i] = z_img[i][s];
      const int64_t cbase = (int64_t)s * V - g.head;
#pragma unroll
      for (int wd = 0; wd < 4; ++wd) {
        float zc[G][N], gc[G][N];
#pragma unroll
        for (int i = 0; i < N; ++i) {
          const uint32_t word = wd == 0 ? rw[i].x : wd == 1 ? rw[i].y : wd == 2 ? rw[i].z : rw[i].w;
          float o[G];
          WordOps<T>::unpack(word, o);
#pragma unroll
          for (int h = 0; h < G; ++h) zc[h][i] = o[h];
        }
#pragma unroll
        for (int h = 0; h < G; ++h) column(zc[h], gc[h], cbase + wd * G + h);
#pragma unroll
        for (int i = 0; i < N; ++i) {
          float o[G];
#pragma unroll
          for (int h = 0; h < G; ++h) o[h] = gc[h][i];
          const uint32_t word = WordOps<T>::pack(o);
          if (wd == 0) rw[i].x = word; else if (wd == 1) rw[i].y = word; else if (wd == 2) rw[i].z = word; else rw[i].w = word;
        }
      }
      if (want_grad) {
#pragma unroll
        for (int i = 0; i < N; ++i)
          reinterpret_cast<uint4*>(reinterpret_cast<T*>(a.grad[i]) + row_off - g.head)[s] = rw[i];
      }
    }
    if (edge) {
#pragma unroll
      for (int e = 0; e < V; ++e) {
        const int64_t c = (int64_t)edge_seg * V - g.head + e;
        if (c < 0 || c >= C) continue;
        float zc[N], gc[N];
#pragma unroll
        for (int i = 0; i < N; ++i) zc[i] = Elem<T>::to_f32(z_row[i][c]);
        column(zc, gc, c);
        if (want_grad) {
#pragma unroll
          for (int i = 0; i < N; ++i) (reinterpret_cast<T*>(a.grad[i]) + row_off)[c] = Elem<T>::from_f32(gc[i]);
        }
      }
    }

    // ================= row results: per-warp distance partials, then lanes 0..n-1 of warp 0 finish the n models
#pragma unroll
    for (int i = 0; i < N; ++i) {
      float dv = dist[i];
      if constexpr (kPackedB) dv += dist2[i].x + dist2[i].y;
      if constexpr (PW && !KL) {   // sum_{j != i} (z_i - z_j)^2 = n z'_i^2 + sum_j z'_j^2, the second sum from all models' z'^2
        float qv = 0.f;
#pragma unroll
        for (int j = 0; j < N; ++j) {
          qv += dist[j];
          if constexpr (kPackedB) qv += dist2[j].x + dist2[j].y;
        }
        dv = fmaf((float)N, dv, qv);
      }
      const float dw = warp_sum(dv);
      if (lane == 0) sh.dist[par][i][warp] = dw;
    }
    __syncthreads();
    if (warp == 0 && lane < N) {
      float dsum = 0.f;
      for (int wv = 0; wv < NW; ++wv) dsum += sh.dist[par][lane][wv];
      const AllRowStat st = sh.stat[par][lane];
      const float ce = (st.m + logf(st.S)) - (1.f - a.eps) * st.zy - (a.eps * inv_C) * st.sum_z;
      // pairwise: 1/((n-1) C) sum_c sum_{j != i} (z_i - z_j)^2;  mean target: 1/C sum_c (kRatio z'_i)^2
      // KL: T^2 / (n-1) sum_{j != i} KL(t_j || t_i)
      const float D = KL ? a.temperature * a.temperature * dsum / (float)(N - 1)
                         : PW ? dsum * inv_C / (float)(N - 1) : dsum * kRatio * kRatio * inv_C;
      uint32_t flags = (st.a_own == y) ? 1u : 0u;
      int bit = 1;
      for (int j = 0; j < N; ++j) {
        if (j == lane) continue;
        if (sh.stat[par][j].a_own == st.a_own) flags |= (1u << bit);
        ++bit;
      }
      a.row_loss[(int64_t)lane * R + r] = with_term ? fmaf(a.alpha, D, ce) : ce;
      a.row_flags[(int64_t)lane * R + r] = flags;
    }
    ++v;
  }

  // ---------------- all rows of this CTA are written: scheduler reset (the final reduction is a kernel of its own)
  stream_last_cta(a.hdr, &sh.last_flag, tid);
}

// Final reduction of the n models: block i sums model i's row losses and counts its flag bits.
__global__ void __launch_bounds__(1024) finalize_all_kernel(const __grid_constant__ AllArgs a) {
  __shared__ double sh[32];
  const int i = blockIdx.x;
  KArgs k = {};
  k.row_loss = a.row_loss + (int64_t)i * a.rows;
  k.row_flags = a.row_flags + (int64_t)i * a.rows;
  k.hdr = a.hdr;
  k.partials = a.partials;
  k.reduced_loss = a.reduced_loss + i;
  k.counters = a.counters ? a.counters + (int64_t)i * (CODISTILL_COUNTERS_FIXED + a.n - 1) : nullptr;
  k.dev_status = i == 0 ? a.dev_status : nullptr;
  k.rows_total = a.rows;
  k.reduction = a.reduction;
  k.n_peers = a.n - 1;
  finalize_cta(k, sh);
}

// ------------------------------------------------------------------ host side
cudaError_t launch_prep_rows(WsHeader* hdr, int64_t* partials, const int32_t* labels, const uint8_t* mask, int64_t rows,
                             int64_t classes, cudaStream_t stream);

struct AllLayout { size_t partials, row_flags, row_loss, total; };
static AllLayout all_layout(int n, int64_t rows) {
  AllLayout l;
  const size_t per = round256(sizeof(uint32_t) * (size_t)n * (size_t)(rows > 0 ? rows : 1));
  l.partials = sizeof(WsHeader);
  l.row_flags = l.partials + round256(sizeof(int64_t) * 2 * kPrepMaxBlocks);
  l.row_loss = l.row_flags + per;
  l.total = l.row_loss + per;
  return l;
}

template <typename T, int N>
static cudaError_t all_launch_n(const AllArgs& a, int num_sms, cudaStream_t stream) {
  const int64_t slots = (int64_t)num_sms * all_ctas_per_sm(N, a.temperature > 0.f);
  const int grid = (int)(a.rows < slots ? a.rows : slots);
  cudaError_t e;
  if (a.temperature > 0.f)  // KL distance, pairwise over the peers
    e = launch_overlapped(rows_all_kernel<T, N, true, true>, dim3(grid), dim3(all_threads(N)), 0, stream, a);
  else if (a.peer_reduce == CODISTILL_PEERS_PAIRWISE_MEAN)
    e = launch_overlapped(rows_all_kernel<T, N, true, false>, dim3(grid), dim3(all_threads(N)), 0, stream, a);
  else
    e = launch_overlapped(rows_all_kernel<T, N, false, false>, dim3(grid), dim3(all_threads(N)), 0, stream, a);
  return e != cudaSuccess ? e : cudaGetLastError();
}

template <typename T>
static cudaError_t all_launch(const AllArgs& a, int num_sms, cudaStream_t stream) {
  switch (a.n) {
    case 2: return all_launch_n<T, 2>(a, num_sms, stream);
    case 3: return all_launch_n<T, 3>(a, num_sms, stream);
    case 4: return all_launch_n<T, 4>(a, num_sms, stream);
    case 5: return all_launch_n<T, 5>(a, num_sms, stream);
    case 6: return all_launch_n<T, 6>(a, num_sms, stream);
    case 7: return all_launch_n<T, 7>(a, num_sms, stream);
    case 8: return all_launch_n<T, 8>(a, num_sms, stream);
    default: return cudaErrorNotSupported;
  }
}

}  // namespace codistill

using namespace codistill;

extern "C" size_t codistill_all_workspace_bytes(int n, int64_t rows) {
  if (n < 2 || n > kAllMax || rows < 0) return 0;
  return all_layout(n, rows).total;
}

extern "C" int codistill_loss_fwd_bwd_all(const codistill_all_params_t* p, void* stream_v) {
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  if (p == nullptr) return CODISTILL_ERR_NULL;
  if (p->struct_bytes != sizeof(codistill_all_params_t)) return CODISTILL_ERR_PARAM;
  if (p->n < 2 || p->n > kAllMax) return CODISTILL_ERR_UNSUPPORTED;
  if (p->rows < 0 || p->classes < 1 || p->row_stride < p->classes) return CODISTILL_ERR_SHAPE;
  if (p->classes > (int64_t)1 << 24 || p->rows > (int64_t)1 << 31) return CODISTILL_ERR_SHAPE;
  if (p->dtype != CODISTILL_F32 && p->dtype != CODISTILL_BF16) return CODISTILL_ERR_DTYPE;
  if (!isfinite(p->alpha) || !(p->label_smoothing >= 0.f && p->label_smoothing < 1.f)) return CODISTILL_ERR_PARAM;
  if (p->peer_reduce != CODISTILL_PEERS_PAIRWISE_MEAN && p->peer_reduce != CODISTILL_PEERS_MEAN_TARGET) return CODISTILL_ERR_PARAM;
  if (p->reduction != CODISTILL_REDUCE_MEAN_VALID && p->reduction != CODISTILL_REDUCE_SUM) return CODISTILL_ERR_PARAM;
  if (p->dist_kind != CODISTILL_DIST_MSE_LOGITS && p->dist_kind != CODISTILL_DIST_MSE_CENTRED &&
      p->dist_kind != CODISTILL_DIST_KL_SOFTMAX)
    return CODISTILL_ERR_UNSUPPORTED;
  if (p->dist_kind == CODISTILL_DIST_KL_SOFTMAX) {
    if (!(p->temperature > 0.f) || !isfinite(p->temperature)) return CODISTILL_ERR_PARAM;
    // the KL form is served pairwise over the peers (for n = 2 the mean target is the same thing)
    if (p->peer_reduce != CODISTILL_PEERS_PAIRWISE_MEAN && p->n != 2) return CODISTILL_ERR_UNSUPPORTED;
  }
  if (p->reduced_loss == nullptr || p->logits == nullptr) return CODISTILL_ERR_NULL;
  if (p->rows > 0 && p->labels == nullptr) return CODISTILL_ERR_NULL;
  uintptr_t bits = 0;
  for (int i = 0; i < p->n; ++i) {
    if (p->rows > 0 && p->logits[i] == nullptr) return CODISTILL_ERR_NULL;
    bits |= reinterpret_cast<uintptr_t>(p->logits[i]);
    if (p->grad_logits) {
      if (p->rows > 0 && p->grad_logits[i] == nullptr) return CODISTILL_ERR_NULL;
      bits |= reinterpret_cast<uintptr_t>(p->grad_logits[i]);
    }
  }
  if (bits & 15u) return CODISTILL_ERR_UNSUPPORTED;  // the 16-byte loads need aligned tensor bases
  if (p->workspace == nullptr || (reinterpret_cast<uintptr_t>(p->workspace) & 255u) != 0) return CODISTILL_ERR_WORKSPACE;
  const AllLayout l = all_layout(p->n, p->rows);
  if (p->workspace_bytes < l.total) return CODISTILL_ERR_WORKSPACE;

  int dev = 0, num_sms = 0, smem_optin = 0;
  if (const int rc_cuda = cuda_status(cudaGetDevice(&dev))) return rc_cuda;
  if (const int rc_cuda = cuda_status(cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, dev))) return rc_cuda;
  if (const int rc_cuda = cuda_status(cudaDeviceGetAttribute(&smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev))) return rc_cuda;

  char* ws = static_cast<char*>(p->workspace);
  AllArgs a;
  memset(&a, 0, sizeof(a));
  for (int i = 0; i < p->n; ++i) { a.model[i] = p->logits[i]; a.grad[i] = p->grad_logits ? p->grad_logits[i] : nullptr; }
  a.labels = p->labels;
  a.mask = p->mask;
  a.row_loss = p->row_loss ? p->row_loss : reinterpret_cast<float*>(ws + l.row_loss);
  a.row_flags = reinterpret_cast<uint32_t*>(ws + l.row_flags);
  a.hdr = reinterpret_cast<WsHeader*>(ws);
  a.partials = reinterpret_cast<const int64_t*>(ws + l.partials);
  a.reduced_loss = p->reduced_loss;
  a.counters = p->counters;
  a.dev_status = p->dev_status;
  a.rows = p->rows;
  a.classes = p->classes;
  a.row_stride = p->row_stride;
  a.n = p->n;
  a.peer_reduce = p->peer_reduce;
  a.reduction = p->reduction;
  a.centred = p->dist_kind == CODISTILL_DIST_MSE_CENTRED;
  a.alpha = p->alpha;
  a.eps = p->label_smoothing;
  a.temperature = p->dist_kind == CODISTILL_DIST_KL_SOFTMAX ? p->temperature : 0.f;  // 0: one of the MSE forms

  if (const int rc_cuda = cuda_status(launch_prep_rows(a.hdr, const_cast<int64_t*>(a.partials), a.labels, a.mask, a.rows, a.classes, stream))) return rc_cuda;
  if (a.rows > 0) {
    // On request (CODISTILL_REGIME=cluster) long rows go to the cluster-resident kernel, which reads every
    // logit from HBM once (the n row images of a row index stay in the shared memory of a cluster) where the
    // direct-load kernel above reads them twice; it is the slower of the two at present (bound by instruction
    // issue, not by memory), so it is not the default.
    const char* want = getenv("CODISTILL_REGIME");
    const bool use_cluster = want != nullptr && strcmp(want, "cluster") == 0;
    cudaError_t e;
    if (use_cluster && cluster_fits(p->n, p->classes, p->row_stride, p->dtype, smem_optin)) {
      ClArgs c;
      memset(&c, 0, sizeof(c));
      for (int i = 0; i < p->n; ++i) { c.model[i] = a.model[i]; c.grad[i] = a.grad[i]; }
      c.labels = a.labels;
      c.mask = a.mask;
      c.row_loss = a.row_loss;
      c.row_flags = a.row_flags;
      c.hdr = a.hdr;
      c.partials = a.partials;
      c.rows_total = a.rows;
      c.row_begin = 0;
      c.row_end = a.rows;
      c.classes = a.classes;
      c.row_stride = a.row_stride;
      c.n = a.n;
      c.pairwise = a.peer_reduce == CODISTILL_PEERS_PAIRWISE_MEAN;
      c.reduction = a.reduction;
      c.centred = a.centred;
      c.alpha = a.alpha;
      c.eps = a.eps;
      c.temperature = p->dist_kind == CODISTILL_DIST_KL_SOFTMAX ? p->temperature : 1.f;
      e = launch_cluster(c, p->dtype, p->dist_kind == CODISTILL_DIST_KL_SOFTMAX ? kClKlPairwise : kClMse, true, smem_optin, stream);
    } else {
      e = p->dtype == CODISTILL_F32 ? all_launch<float>(a, num_sms, stream) : all_launch<__nv_bfloat16>(a, num_sms, stream);
    }
    if (const int rc_cuda = cuda_status(e)) return rc_cuda;
  }
  finalize_all_kernel<<<a.n, 1024, 0, stream>>>(a);
  return cuda_status(cudaGetLastError());
}
