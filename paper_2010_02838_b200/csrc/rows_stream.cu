// Streaming kernel for long rows ("stream" regime), MSE-on-logits distance.
//
// One CTA of 256 (many peers: 128) threads works on one row at a time; several CTAs are resident per SM and draw rows
// from a global counter.  Nothing is staged in shared memory.  Every thread reads its 16-byte
// segments of the row straight from global memory, several loads in flight per thread:
//   pass A  the own row once: online softmax (running maximum with its first segment, sum exp,
//           sum z), then one block reduction gives the row statistics;
//   pass B  the own row again, together with the n-1 peer rows: differences, squared distance,
//           what the arg-max agreement needs, the gradient, written with 16-byte stores.
// The second read of the own row comes a few microseconds after the first and is served by the
// L2 cache, so that HBM sees every logit once and the gradient once, as in the staged kernel.
// With no shared-memory row buffer the row length is unbounded: this kernel serves the rows that are
// too long for the staged kernel (vocabularies beyond about 90 K bf16 classes).
//
// Rows need not be 16-byte aligned: a thread works on the segments of the row image (the aligned
// byte range that holds the row) that lie wholly inside the row; the ragged first / last segments
// of an unaligned row are done element by element by two designated threads.
#include <type_traits>


#include "stream_common.cuh"

namespace codistill {

// CEN: the centred distance (logits minus their class means): one more pass sums every peer row first.
template <typename T, int P, bool PW, bool CEN>
__global__ void __launch_bounds__(stream_threads(P), stream_ctas_per_sm(P)) rows_stream_kernel(const __grid_constant__ KArgs a) {
  constexpr int V = SegOps<T>::V;
  constexpr int H = SegOps<T>::H;
  constexpr int PD = P > 0 ? P : 1;
  constexpr int NT = stream_threads(P);
  constexpr int kAhead = stream_ahead(P);
  constexpr int kStreamWarps = NT / 32;
  __shared__ StreamShared sh;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t C = a.classes;
  const bool with_term = (P >= 1 && a.alpha != 0.f);
  const bool stream_peers = (P >= 1) && (with_term || a.want_flags);

  wait_for_prior_grid();  // from here on the workspace header and the valid-row counts are read
#if STREAM_HINTS
  const uint64_t pol_keep = make_policy_keep(), pol_stream = make_policy_stream();
#endif
  float w = 1.f;
  if (a.reduction == CODISTILL_REDUCE_MEAN_VALID) {
    const int64_t nv = total_valid(a);
    w = 1.f / (float)(nv > 1 ? nv : 1);
  }
  const float inv_P = P >= 1 ? 1.f / (float)P : 0.f;
  const float inv_C = 1.f / (float)C;
  const float2 l2e2 = make_float2(kLog2e, kLog2e);
  const float2 neg1 = make_float2(-1.f, -1.f);

  stream_draw_row(&sh.next_row[0], a.hdr, a.row_begin, tid);
  __syncthreads();
  int v = 0;  // valid rows done by this CTA
  for (int it = 0;; ++it) {
    const long long r = sh.next_row[it & 1];
    if (r >= a.row_end) break;
    stream_draw_row(&sh.next_row[(it + 1) & 1], a.hdr, a.row_begin, tid);
    const StreamRow row = stream_row<T, NT>(r - a.row_begin, r, a.row_stride, C, a.labels, a.mask, tid);
    const RowGeom g = row.g;
    const int64_t row_off = row.row_off;  // in elements
    const T* __restrict__ z_row = reinterpret_cast<const T*>(a.own) + row_off;
    T* __restrict__ g_row = a.grad ? reinterpret_cast<T*>(a.grad) + row_off : nullptr;
    const uint4* __restrict__ z_img = reinterpret_cast<const uint4*>(z_row - g.head);
    uint4* __restrict__ g_img = g_row ? reinterpret_cast<uint4*>(g_row - g.head) : nullptr;
    const int cnt = row.cnt, s0 = row.s0, y = row.y;
    const bool edge_head = row.edge_head, edge_tail = row.edge_tail;

    if (!row.valid) {  // masked row: zero gradient, no loss, no counts; nothing is read
      if (g_row) stream_zero_row<T, NT>(g_row, row, C);
      if (tid == 0) { a.row_loss[r] = 0.f; a.row_flags[r] = 0u; }
      __syncthreads();  // orders the row-id hand-over
      continue;
    }
    const int par = v & 1;

    // ================= pass A: own-row statistics
    float best = -3.0e38f;  // finite, so that the first rescale is exp2(-huge) = 0 and never NaN
    int best_seg = 0x7fffffff;
    float2 s2[H], zs2[H];
#pragma unroll
    for (int i = 0; i < H; ++i) { s2[i] = make_float2(0.f, 0.f); zs2[i] = make_float2(0.f, 0.f); }
    float s_edge = 0.f, z_edge = 0.f;
    auto sweep_batch = [&](auto nb, int i0) {
      constexpr int B = decltype(nb)::value;
      if (kAhead > 0) {
#pragma unroll
        for (int u = 0; u < B; ++u) {
          const int ia = i0 + kAhead * B + u;
          if (ia < cnt) prefetch_l2(z_img + s0 + ia * NT);
        }
      }
      uint4 rw[B];
#pragma unroll
#if STREAM_HINTS & 1
      for (int u = 0; u < B; ++u) rw[u] = ldg_policy(z_img + s0 + (i0 + u) * NT, pol_keep);
#else
      for (int u = 0; u < B; ++u) rw[u] = z_img[s0 + (i0 + u) * NT];
#endif
      const float old_best = best;
#pragma unroll
      for (int u = 0; u < B; ++u) {
        const float fm = SegOps<T>::to_float(SegOps<T>::fold(rw[u]));
        if (fm > best) { best = fm; best_seg = s0 + (i0 + u) * NT; }
      }
      const float sc = rescale_exp2<T>((old_best - best) * kLog2e);
      const float2 sc2 = make_float2(sc, sc);
      const float2 nmk = make_float2(-best * kLog2e, -best * kLog2e);
      s_edge *= sc;
#pragma unroll
      for (int i = 0; i < H; ++i) s2[i] = __fmul2_rn(s2[i], sc2);
#pragma unroll
      for (int u = 0; u < B; ++u) {
        float2 z2[H];
        SegOps<T>::unpack2(rw[u], z2);
#pragma unroll
        for (int i = 0; i < H; ++i) {
          s2[i] = __fadd2_rn(s2[i], exp_shift2<T>(z2[i], best, l2e2, nmk));
          zs2[i] = __fadd2_rn(zs2[i], z2[i]);
        }
      }
    };
    {
      int i = 0;
      for (; i + kBatchA <= cnt; i += kBatchA) sweep_batch(std::integral_constant<int, kBatchA>{}, i);
      for (; i < cnt; ++i) sweep_batch(std::integral_constant<int, 1>{}, i);
    }
    if (edge_head || edge_tail) {  // ragged segment, element by element
      const int s = edge_head ? 0 : g.n_seg - 1;
      float zv[V];
      float fm = -3.0e38f;
#pragma unroll
      for (int i = 0; i < V; ++i) {
        const int64_t c = (int64_t)s * V - g.head + i;
        zv[i] = (c >= 0 && c < C) ? Elem<T>::to_f32(z_row[c]) : -INFINITY;
        fm = fmaxf(fm, zv[i]);
      }
      const float old_best = best;
      if (fm > best || (fm == best && s < best_seg)) { best = fm; best_seg = s; }
      const float sc = rescale_exp2<T>((old_best - best) * kLog2e);
      const float2 sc2 = make_float2(sc, sc);
      const float2 nmk = make_float2(-best * kLog2e, -best * kLog2e);
      s_edge *= sc;
#pragma unroll
      for (int i = 0; i < H; ++i) s2[i] = __fmul2_rn(s2[i], sc2);
#pragma unroll
      for (int i = 0; i < V; ++i) {
        if (zv[i] != -INFINITY) {
          s_edge += exp_shift2<T>(make_float2(zv[i], zv[i]), best, l2e2, nmk).x;
          z_edge += zv[i];
        }
      }
    }
    float s_t = s_edge, z_t = z_edge;
#pragma unroll
    for (int i = 0; i < H; ++i) { s_t += s2[i].x + s2[i].y; z_t += zs2[i].x + zs2[i].y; }
    // block reduction in one round: maximum with its first segment, then the sums rescaled to it
    float m;
    int m_seg;
    float S = 0.f, sum_z = 0.f;
    {
      const unsigned key = float_order_key(best + 0.f);  // -0 is folded onto +0: they tie
      const unsigned key_w = __reduce_max_sync(0xffffffffu, key);
      const int seg_w = (int)__reduce_min_sync(0xffffffffu, key == key_w ? (unsigned)best_seg : 0x7fffffffu);
      const float m_w = float_from_order_key(key_w);
      const float sw = warp_sum(s_t * rescale_exp2<T>((best - m_w) * kLog2e));
      const float zw = warp_sum(z_t);
      if (lane == 0) sh.red[par][warp] = make_float4(m_w, __int_as_float(seg_w), sw, zw);
      __syncthreads();
      float4 part[kStreamWarps];
#pragma unroll
      for (int wv = 0; wv < kStreamWarps; ++wv) part[wv] = sh.red[par][wv];
      m = part[0].x;
      m_seg = __float_as_int(part[0].y);
#pragma unroll
      for (int wv = 1; wv < kStreamWarps; ++wv) argmax_combine(m, m_seg, part[wv].x, __float_as_int(part[wv].y));
#pragma unroll
      for (int wv = 0; wv < kStreamWarps; ++wv) {
        S += part[wv].z * rescale_exp2<T>((part[wv].x - m) * kLog2e);
        sum_z += part[wv].w;
      }
    }
    if (m_seg >= g.n_seg) m_seg = 0;  // NaN rows: keep the reads below inside the row
    const int a_own = first_equal_global<T>(z_row, m_seg, g.head, C, m);
    const int seg_a = a.want_flags ? m_seg : -1;
    const float zy = Elem<T>::to_f32(z_row[y]);

    // ================= pass B: peers, distance, gradient
    const float2 nml2 = make_float2(-m * kLog2e, -m * kLog2e);
    const float cp = w * __frcp_rn(S);                                          // e_c -> w * p_c
    const float cd = with_term ? w * a.alpha * (2.f * inv_C) * inv_P : 0.f;     // sum_j d -> w * alpha * dD
    const float cq = w * a.eps * inv_C;
    const float cy = w * (1.f - a.eps);
    const float2 cp2 = make_float2(cp, cp), cd2 = make_float2(cd, cd), ncq2 = make_float2(-cq, -cq);
    const int seg_y = (g.head + y) / V, pos_y = (g.head + y) % V;
    float2 dist2 = make_float2(0.f, 0.f), dist2b = make_float2(0.f, 0.f);
    typename SegOps<T>::macc lt[PD], ge[PD];
    float za[PD];
#pragma unroll
    for (int j = 0; j < PD; ++j) { lt[j] = SegOps<T>::neg_inf(); ge[j] = SegOps<T>::neg_inf(); za[j] = -INFINITY; }
    const uint4* p_img[PD];
#pragma unroll
    for (int j = 0; j < PD; ++j)
      p_img[j] = P > 0 ? reinterpret_cast<const uint4*>(reinterpret_cast<const T*>(a.peers[j]) + row_off - g.head) : nullptr;

    // centred distance: d_j = (z - mean z) - (v_j - mean v_j) = (z - v_j) - shift_j, shift_j = mean z - mean v_j
    float2 nshift2[PD];
    float shift[PD];
#pragma unroll
    for (int j = 0; j < PD; ++j) { shift[j] = 0.f; nshift2[j] = make_float2(0.f, 0.f); }
    if constexpr (CEN && P > 0) {
      if (with_term) {
        float2 ps2[PD];
        float pe[PD];
#pragma unroll
        for (int j = 0; j < PD; ++j) { ps2[j] = make_float2(0.f, 0.f); pe[j] = 0.f; }
        for (int i0 = 0; i0 < cnt; ++i0) {
          if (kAhead > 0 && i0 + 4 < cnt) {   // the peers' segments four iterations on: into the L2
#pragma unroll
            for (int j = 0; j < P; ++j) prefetch_l2(p_img[j] + s0 + (i0 + 4) * NT);
          }
          uint4 pr[PD];
#pragma unroll
          for (int j = 0; j < P; ++j) pr[j] = ldg_policy(p_img[j] + s0 + i0 * NT, pol_keep);
#pragma unroll
          for (int j = 0; j < P; ++j) {
            float2 v2[H];
            SegOps<T>::unpack2(pr[j], v2);
#pragma unroll
            for (int i = 0; i < H; ++i) ps2[j] = __fadd2_rn(ps2[j], v2[i]);
          }
        }
        if (edge_head || edge_tail) {
          const int s = edge_head ? 0 : g.n_seg - 1;
#pragma unroll
          for (int i = 0; i < V; ++i) {
            const int64_t c = (int64_t)s * V - g.head + i;
            if (c < 0 || c >= C) continue;
#pragma unroll
            for (int j = 0; j < P; ++j) pe[j] += Elem<T>::to_f32(reinterpret_cast<const T*>(a.peers[j])[row_off + c]);
          }
        }
#pragma unroll
        for (int j = 0; j < P; ++j) {
          const float sw = warp_sum(ps2[j].x + ps2[j].y + pe[j]);
          if (lane == 0) sh.cen[par][j][warp] = sw;
        }
        __syncthreads();
#pragma unroll
        for (int j = 0; j < P; ++j) {
          float tot = 0.f;
#pragma unroll
          for (int wv = 0; wv < kStreamWarps; ++wv) tot += sh.cen[par][j][wv];
          shift[j] = (sum_z - tot) * inv_C;
          nshift2[j] = make_float2(-shift[j], -shift[j]);
        }
      }
    }

    auto grad_batch = [&](auto nb, int i0) {
      constexpr int B = decltype(nb)::value;
      if (kAhead > 0 && stream_peers) {  // the peers' segments of a later batch: into the L2, no register held
#pragma unroll
        for (int u = 0; u < B; ++u) {
          const int ia = i0 + kAhead * B + u;
          if (ia < cnt) {
#pragma unroll
            for (int j = 0; j < P; ++j) prefetch_l2(p_img[j] + s0 + ia * NT);
          }
        }
      }
      uint4 zr[B];
#pragma unroll
      for (int u = 0; u < B; ++u) zr[u] = z_img[s0 + (i0 + u) * NT];
      float2 z2[B][H], sd2[B][H];
#pragma unroll
      for (int u = 0; u < B; ++u) {
#pragma unroll
        for (int i = 0; i < H; ++i) sd2[u][i] = make_float2(0.f, 0.f);
      }
      if (stream_peers) {
#pragma unroll
        for (int u = 0; u < B; ++u) SegOps<T>::unpack2(zr[u], z2[u]);
        constexpr int PG = PD;
#pragma unroll
        for (int j0 = 0; j0 < P; j0 += PG) {
        uint4 pr[PG][B];
#pragma unroll
        for (int jj = 0; jj < PG; ++jj) {
          if (j0 + jj < P) {
#pragma unroll
#if STREAM_HINTS & 2
            for (int u = 0; u < B; ++u) pr[jj][u] = ldg_policy(p_img[j0 + jj] + s0 + (i0 + u) * NT, pol_stream);
#else
            for (int u = 0; u < B; ++u) pr[jj][u] = p_img[j0 + jj][s0 + (i0 + u) * NT];
#endif
          }
        }
#pragma unroll
        for (int jj = 0; jj < PG; ++jj) {
          const int j = j0 + jj;
          if (j >= P) break;
#pragma unroll
          for (int u = 0; u < B; ++u) {
            const int s = s0 + (i0 + u) * NT;
            float2 v2[H];
            SegOps<T>::unpack2(pr[jj][u], v2);
#pragma unroll
            for (int i = 0; i < H; ++i) {
              const float2 d = CEN ? __ffma2_rn(v2[i], neg1, __fadd2_rn(z2[u][i], nshift2[j])) : __ffma2_rn(v2[i], neg1, z2[u][i]);
              if (P == 1 || j == 0) sd2[u][i] = d; else sd2[u][i] = __fadd2_rn(sd2[u][i], d);
              if constexpr (PW) { if (i & 1) dist2b = __ffma2_rn(d, d, dist2b); else dist2 = __ffma2_rn(d, d, dist2); }
            }
            const typename SegOps<T>::macc f = SegOps<T>::fold(pr[jj][u]);
            const bool before = s < seg_a;
            lt[j] = before ? SegOps<T>::mmax(lt[j], f) : lt[j];
            ge[j] = before ? ge[j] : SegOps<T>::mmax(ge[j], f);
            if (s == seg_a) {
              // The segment of the own arg-max column a went to ge[] as a whole.  The peer's value at a and
              // the largest value before a inside the segment settle the rest: with them in za[] and lt[],
              // "za >= ge and lt < za" holds exactly when the peer's first arg-max is a.
              float vv[V];
              SegOps<T>::unpack(pr[jj][u], vv);
              float pre = -INFINITY;
#pragma unroll
              for (int i = 0; i < V; ++i) {
                const int c = seg_a * V - g.head + i;
                if (c < a_own) pre = fmaxf(pre, vv[i]);
                if (c == a_own) za[j] = vv[i];
              }
              lt[j] = SegOps<T>::mmax(lt[j], SegOps<T>::from_scalar(pre));
            }
          }
        }
        }
      } else {
#pragma unroll
        for (int u = 0; u < B; ++u) SegOps<T>::unpack2(zr[u], z2[u]);
      }
#pragma unroll
      for (int u = 0; u < B; ++u) {
        const int s = s0 + (i0 + u) * NT;
        float2 g2[H];
#pragma unroll
        for (int i = 0; i < H; ++i) {
          const float2 e = exp_shift2<T>(z2[u][i], m, l2e2, nml2);
          g2[i] = __ffma2_rn(e, cp2, __ffma2_rn(sd2[u][i], cd2, ncq2));
          if constexpr (!PW) dist2 = __ffma2_rn(sd2[u][i], sd2[u][i], dist2);  // (sum_j d)^2, scaled by 1/P^2 below
        }
        if (s == seg_y) {  // the label column: q_y carries the extra 1 - eps
#pragma unroll
          for (int i = 0; i < H; ++i) {
            if (2 * i == pos_y) g2[i].x -= cy;
            if (2 * i + 1 == pos_y) g2[i].y -= cy;
          }
        }
#if STREAM_HINTS & 4
        if (g_img) stg_policy(g_img + s, SegOps<T>::pack2(g2), pol_stream);
#else
        if (g_img) g_img[s] = SegOps<T>::pack2(g2);
#endif
      }
    };
    {
      int i = 0;
      constexpr int BB = P >= 3 ? 1 : kBatchB;
      for (; i + BB <= cnt; i += BB) grad_batch(std::integral_constant<int, BB>{}, i);
      for (; i < cnt; ++i) grad_batch(std::integral_constant<int, 1>{}, i);
    }
    float dist_edge = 0.f;
    if (edge_head || edge_tail) {  // ragged segment, element by element
      const int s = edge_head ? 0 : g.n_seg - 1;
#pragma unroll
      for (int i = 0; i < V; ++i) {
        const int64_t c = (int64_t)s * V - g.head + i;
        if (c < 0 || c >= C) continue;
        const float z = Elem<T>::to_f32(z_row[c]);
        float sd = 0.f;
        if (stream_peers) {
#pragma unroll
          for (int j = 0; j < P; ++j) {
            const float pv = Elem<T>::to_f32(reinterpret_cast<const T*>(a.peers[j])[row_off + c]);
            const float d = (z - pv) - shift[j];
            sd += d;
            if constexpr (PW) dist_edge = fmaf(d, d, dist_edge);
            if (a.want_flags) {
              if (c < a_own) lt[j] = SegOps<T>::mmax(lt[j], SegOps<T>::from_scalar(pv));
              else if (c > a_own) ge[j] = SegOps<T>::mmax(ge[j], SegOps<T>::from_scalar(pv));
              else za[j] = pv;
            }
          }
        }
        if constexpr (!PW) dist_edge = fmaf(sd, sd, dist_edge);
        const float e = exp_shift2<T>(make_float2(z, z), m, l2e2, nml2).x;
        float gv = fmaf(e, cp, fmaf(sd, cd, -cq));
        if (c == (int64_t)y) gv -= cy;
        if (g_row) g_row[c] = Elem<T>::from_f32(gv);
      }
    }

    // ================= row results: per-warp partials, then warp 0 finishes the row
    {
      float part[1 + 3 * PD];
      part[0] = warp_sum((dist2.x + dist2.y) + (dist2b.x + dist2b.y) + dist_edge);
#pragma unroll
      for (int j = 0; j < PD; ++j) {
        part[1 + 3 * j] = warp_max_redux(SegOps<T>::to_float(lt[j]));
        part[2 + 3 * j] = warp_max_redux(SegOps<T>::to_float(ge[j]));
        part[3 + 3 * j] = warp_max_redux(za[j]);
      }
      if (lane == 0) {
#pragma unroll
        for (int i = 0; i < 1 + 3 * PD; ++i) sh.endred[par][i * kStreamWarps + warp] = part[i];
      }
      __syncthreads();
      if (warp == 0) {
        const float* er = sh.endred[par];
        const float dsum = warp_sum(lane < kStreamWarps ? er[lane] : 0.f);
        uint32_t flags = 0u;
        if (a.want_flags) {
          flags = (a_own == y) ? 1u : 0u;
#pragma unroll
          for (int j = 0; j < P; ++j) {
            const float ltv = warp_max_redux(lane < kStreamWarps ? er[(1 + 3 * j) * kStreamWarps + lane] : -INFINITY);
            const float gev = warp_max_redux(lane < kStreamWarps ? er[(2 + 3 * j) * kStreamWarps + lane] : -INFINITY);
            const float zav = warp_max_redux(lane < kStreamWarps ? er[(3 + 3 * j) * kStreamWarps + lane] : -INFINITY);
            if (zav >= gev && ltv < zav) flags |= (2u << j);
          }
        }
        if (lane == 0) {
          const float ce = (m + logf(S)) - (1.f - a.eps) * zy - (a.eps * inv_C) * sum_z;
          float D = 0.f;
          if (with_term) D = PW ? dsum * inv_P * inv_C : dsum * inv_P * inv_P * inv_C;
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
cudaError_t launch_stream_kl(const KArgs& a, int dtype, int num_sms, cudaStream_t stream);

bool stream_supported(const KArgs& a, int dtype) {
  const int64_t es = dtype == CODISTILL_F32 ? 4 : 2;
  if (a.dist != CODISTILL_DIST_MSE_LOGITS && a.dist != CODISTILL_DIST_KL_SOFTMAX && a.dist != CODISTILL_DIST_MSE_CENTRED) return false;
  if (!(a.n_peers == 0 || a.n_peers == 1 || a.n_peers == 2 || a.n_peers == 3 || a.n_peers == 7)) return false;
  if (a.classes * es < 8192 || a.classes > (int64_t)1 << 24) return false;
  uintptr_t bits = reinterpret_cast<uintptr_t>(a.own) | reinterpret_cast<uintptr_t>(a.grad);
  for (int j = 0; j < a.n_peers; ++j) bits |= reinterpret_cast<uintptr_t>(a.peers[j]);
  return (bits & 15u) == 0;
}

template <typename T, int P, bool PW>
static cudaError_t stream_launch_one(const KArgs& a, int grid, cudaStream_t stream) {
  cudaError_t e;
  if (a.dist == CODISTILL_DIST_MSE_CENTRED)
    e = launch_overlapped(rows_stream_kernel<T, P, PW, true>, dim3(grid), dim3(stream_threads(P)), 0, stream, a);
  else
    e = launch_overlapped(rows_stream_kernel<T, P, PW, false>, dim3(grid), dim3(stream_threads(P)), 0, stream, a);
  return e != cudaSuccess ? e : cudaGetLastError();
}

template <typename T>
static cudaError_t stream_launch_peers(const KArgs& a, int grid, cudaStream_t stream) {
  const bool pw = a.peer_reduce == CODISTILL_PEERS_PAIRWISE_MEAN;  // with one peer both readings coincide
  switch (a.n_peers) {
    case 0: return stream_launch_one<T, 0, true>(a, grid, stream);
    case 1: return stream_launch_one<T, 1, true>(a, grid, stream);
    case 2: return pw ? stream_launch_one<T, 2, true>(a, grid, stream) : stream_launch_one<T, 2, false>(a, grid, stream);
    case 3: return pw ? stream_launch_one<T, 3, true>(a, grid, stream) : stream_launch_one<T, 3, false>(a, grid, stream);
    case 7: return pw ? stream_launch_one<T, 7, true>(a, grid, stream) : stream_launch_one<T, 7, false>(a, grid, stream);
    default: return cudaErrorNotSupported;
  }
}

cudaError_t launch_stream(const KArgs& a, int dtype, int num_sms, cudaStream_t stream) {
  if (!stream_supported(a, dtype)) return cudaErrorNotSupported;
  if (a.dist == CODISTILL_DIST_KL_SOFTMAX) return launch_stream_kl(a, dtype, num_sms, stream);
  const int64_t rows = a.row_end - a.row_begin;
  if (rows <= 0) return cudaSuccess;
  const int64_t slots = (int64_t)num_sms * stream_ctas_per_sm(a.n_peers);
  const int grid = (int)(rows < slots ? rows : slots);
  return dtype == CODISTILL_F32 ? stream_launch_peers<float>(a, grid, stream) : stream_launch_peers<__nv_bfloat16>(a, grid, stream);
}

}  // namespace codistill
