// Cluster-resident kernel for long rows ("cluster" regime): every logit is read from HBM once.
//
// A thread-block cluster of K CTAs works on one row index at a time.  CTA k of the cluster owns a
// fixed range of the 16-byte segments of the row image and keeps that range of ALL n logit tensors
// (the n codistilled models of Algorithm 1: own + peers) in its shared memory, brought in by 1-D bulk
// asynchronous copies (cp.async.bulk, no multicast) that complete on one mbarrier.  Both passes then
// run from shared memory:
//   pass A  per tensor the online softmax statistics of the CTA's range (maximum with its first
//           column, sum exp, sum z, and for the KL form sum exp at temperature T); the K partial
//           results of a tensor are exchanged through distributed shared memory after one cluster
//           barrier, so that every CTA knows the statistics of the whole row;
//   pass B  column by column over the CTA's range with the n models side by side: distance terms
//           and the gradient of every requested model, written with 16-byte stores.
// The distance partial sums of a row are collected by CTA 0 of the cluster behind the next row's
// cluster barrier (nobody waits for them), which then writes the row's loss and flag word.
//
// Served: the all-models call (model i against the other n-1, all i) and the single-model call
// (model 0 against its peers) with the distances whose gradient needs row statistics of the peers:
// MSE on centred logits and the softmax-KL form, and plain MSE as an option.  The arithmetic is the
// one of rows_all.cu: per column the n logits are centred on their mean over the models,
//   z_i - zbar_(-i) = n/(n-1) z'_i,   sum_{j != i} (z_i - z_j)^2 = n z'_i^2 + sum_j z'_j^2,
// and for KL with t_j = softmax(z_j / T), Q = sum_j t_j, E = sum_j t_j log t_j,
//   sum_{j != i} KL(t_j || t_i) = sum_c (E_c - Q_c log t_ic),   d/dz_ic = T (n t_ic - Q_c) / ... .
// A single-model call is the i = 0 part of the same sums.  The KL distance to the softmax of the
// averaged peer logits (mean target, single-model call only) takes the statistics of that average
// as one more tensor in pass A.
#include <cooperative_groups.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <map>
#include <mutex>
#include <tuple>
#include <type_traits>

#include "bulk_copy.cuh"
#include "cluster_args.cuh"
#include "common.cuh"
#include "seg_math.cuh"

namespace cg = cooperative_groups;

namespace codistill {

constexpr int kClThreads = 256;
constexpr int kClWarps = kClThreads / 32;
constexpr int kClMaxCluster = 16;
constexpr int kClCtrlBytes = 12288;
constexpr uint32_t kClCopyPiece = 32768;
constexpr unsigned long long kClWaitLimitNs = 2000000000ull;   // bounded waits: 2 s, then CODISTILL_DEV_TIMEOUT
constexpr unsigned long long kClDrainLimitNs = 50000000ull;    // last wait of an aborted CTA: 50 ms

// what one warp found in a sub-range of one tensor
struct ClRec { float m; int seg; float S, sum_z, S_T; int tensor; };
// what one CTA found in its range of one tensor
struct ClPart { float m; int col; float S, sum_z, S_T, zy; };   // zy: the label's logit if it lies in the range, else 0
// statistics of a whole row of one tensor
struct ClStat { float m, S, sum_z, S_T, zy; int col; };

struct ClCtrl {
  uint64_t full[kClMax];                   // bulk copies of tensor i's range of the current row have landed
  int abort_flag;
  ClRec rec[kClWarps][kClMax + 1];         // pass A: what warp w found in its share of tensor i (slot n: the averaged peers)
  ClPart gather[2][kClMaxCluster][kClMax + 1];   // [row parity][CTA of the cluster][tensor]: written by that CTA into every CTA
  float dgather[2][kClMaxCluster][kClMax + 1];   // CTA 0: distance partial sums [parity][CTA][model]; slot kClMax: sum_j z'_j^2
  float dwarp[kClWarps][kClMax + 1];
  ClStat stat[kClMax + 1];                 // current row, combined over the cluster
  ClStat pend[2][kClMax + 1];              // CTA 0: statistics of the rows whose loss is still to be written
  long long pend_row[2];
  int pend_y[2];
};
static_assert(sizeof(ClCtrl) <= kClCtrlBytes, "control block fits its slot");

// Wait for a phase of the copy barrier, but never for ever: after the limit the CTA-wide abort flag and the
// device status are set and later waits return early (results are then invalid, control flow stays uniform).
__device__ __forceinline__ void cl_wait(uint64_t* bar, uint32_t parity, ClCtrl* ctrl, WsHeader* hdr) {
  if (mbar_try_wait(bar, parity)) return;
  mbar_wait_limited(bar, parity, &ctrl->abort_flag, &hdr->status, CODISTILL_DEV_TIMEOUT, kClWaitLimitNs, true, true);
}

// exp((z - m) / T) for a pair of columns; l2eT = log2(e) / T
template <typename T>
__device__ __forceinline__ float2 exp_temp2(float2 z, float m, float inv_T, float l2eT) {
  if constexpr (sizeof(T) == 4) {
    return make_float2(expf((z.x - m) * inv_T), expf((z.y - m) * inv_T));
  } else {
    const float2 t = __ffma2_rn(z, make_float2(l2eT, l2eT), make_float2(-m * l2eT, -m * l2eT));
    return make_float2(ex2_approx(t.x), ex2_approx(t.y));
  }
}
// exp(x), x in natural units: full precision for fp32 logits, the hardware exp2 for bf16 logits
template <typename T>
__device__ __forceinline__ float exp_nat1(float x) {
  if constexpr (sizeof(T) == 4) return expf(x); else return ex2_approx(x * kLog2e);
}

// One lane's statistics of its segments of one tensor; the sums are relative to `best`.
struct ClLane { float best; int seg; float s, z, t; };

// Statistics of the lane's share of segments [q_lo, q_hi) of one tensor's range (all of them whole segments
// inside the row), four segments at a time: the maximum of the batch first, then the exponentials against a
// fixed reference -- no branch in the loop body.  Lanes without a segment return best = -3e38, sums 0.
template <typename T, bool TEMP>
__device__ __forceinline__ ClLane cl_sweep_range(const char* sl, int q_lo, int q_hi, int seg_begin, int tid, float inv_T, bool need_z) {
  constexpr int H = SegOps<T>::H;
  constexpr int U = 4;
  constexpr uint32_t kPad = sizeof(T) == 4 ? 0xFF800000u : 0xFF80FF80u;   // -inf in every element: no maximum, exp = 0
  ClLane L;
  L.best = -3.0e38f; L.seg = 0x7fffffff; L.s = 0.f; L.z = 0.f; L.t = 0.f;
  float2 s2[H], t2[H], zs2[H];
#pragma unroll
  for (int h = 0; h < H; ++h) { s2[h] = make_float2(0.f, 0.f); t2[h] = s2[h]; zs2[h] = s2[h]; }
  const float2 l2e2 = make_float2(kLog2e, kLog2e);
#pragma unroll 1
  for (int q = q_lo + tid; q < q_hi; q += U * kClThreads) {
    uint4 raw[U];
    float fm[U];
    bool ok[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int qq = q + u * kClThreads;
      ok[u] = qq < q_hi;
      raw[u] = ok[u] ? *reinterpret_cast<const uint4*>(sl + (size_t)qq * 16) : make_uint4(kPad, kPad, kPad, kPad);
      fm[u] = SegOps<T>::to_float(SegOps<T>::fold(raw[u]));
    }
    const float bm = fmaxf(fmaxf(fm[0], fm[1]), fmaxf(fm[2], fm[3]));
    int sb = seg_begin + q + (U - 1) * kClThreads;   // the first segment of the batch that attains its maximum
#pragma unroll
    for (int u = U - 2; u >= 0; --u) sb = fm[u] == bm ? seg_begin + q + u * kClThreads : sb;
    const float nb = fmaxf(L.best, bm);
    const float sc = rescale_exp2<T>((L.best - nb) * kLog2e);
#pragma unroll
    for (int h = 0; h < H; ++h) s2[h] = __fmul2_rn(s2[h], make_float2(sc, sc));
    if constexpr (TEMP) {
      const float st = rescale_exp2<T>((L.best - nb) * (kLog2e * inv_T));
#pragma unroll
      for (int h = 0; h < H; ++h) t2[h] = __fmul2_rn(t2[h], make_float2(st, st));
    }
    L.seg = bm > L.best ? sb : L.seg;
    L.best = nb;
    const float2 nmk = make_float2(-nb * kLog2e, -nb * kLog2e);
#pragma unroll
    for (int u = 0; u < U; ++u) {
      if (u > 0 && !ok[u]) continue;   // padding: nothing to add (the same for all lanes of most warps)
      float2 z2[H];
      SegOps<T>::unpack2(raw[u], z2);
#pragma unroll
      for (int h = 0; h < H; ++h) {
        s2[h] = __fadd2_rn(s2[h], exp_shift2<T>(z2[h], nb, l2e2, nmk));
        if constexpr (TEMP) t2[h] = __fadd2_rn(t2[h], exp_temp2<T>(z2[h], nb, inv_T, kLog2e * inv_T));
      }
      if (need_z) {   // the sum of the logits: label smoothing and the centred distance only
#pragma unroll
        for (int h = 0; h < H; ++h) zs2[h] = __fadd2_rn(zs2[h], z2[h]);
      }
    }
  }
  float2 sa = s2[0], ta = t2[0], za = zs2[0];
#pragma unroll
  for (int h = 1; h < H; ++h) { sa = __fadd2_rn(sa, s2[h]); ta = __fadd2_rn(ta, t2[h]); za = __fadd2_rn(za, zs2[h]); }
  L.s = sa.x + sa.y;
  L.t = ta.x + ta.y;
  L.z = za.x + za.y;
  return L;
}

// Adds one ragged segment (first or last of the row image: only the columns inside the row count) to a
// lane's statistics.  In and out by value, so that the caller's copy stays in registers.
template <typename T, bool TEMP>
__device__ __noinline__ ClLane cl_sweep_edge(ClLane L, uint4 raw, int s, int head, int64_t C, float inv_T) {
  constexpr int V = SegOps<T>::V;
  float z[V];
  SegOps<T>::unpack(raw, z);
  float fm = -3.0e38f;
#pragma unroll
  for (int e = 0; e < V; ++e) {
    const int64_t c = (int64_t)s * V - head + e;
    if (c >= 0 && c < C) fm = fmaxf(fm, z[e]);
  }
  // the ragged segments are the first or the last of the row: an equal maximum in segment 0 comes first
  const bool take = fm > L.best || (fm == L.best && s < L.seg);
  const float nb = fmaxf(L.best, fm);
  L.s *= rescale_exp2<T>((L.best - nb) * kLog2e);
  if constexpr (TEMP) L.t *= rescale_exp2<T>((L.best - nb) * (kLog2e * inv_T));
  if (take) L.seg = s;
  L.best = nb;
  const float2 l2e2 = make_float2(kLog2e, kLog2e);
  const float2 nmk = make_float2(-nb * kLog2e, -nb * kLog2e);
#pragma unroll
  for (int e = 0; e < V; ++e) {
    const int64_t c = (int64_t)s * V - head + e;
    if (c >= 0 && c < C) {
      L.s += exp_shift2<T>(make_float2(z[e], z[e]), nb, l2e2, nmk).x;
      L.z += z[e];
      if constexpr (TEMP) L.t += exp_temp2<T>(make_float2(z[e], z[e]), nb, inv_T, kLog2e * inv_T).x;
    }
  }
  return L;
}

// Sums NV per-lane values (NV a power of two, 2..32) across the warp in NV - 1 + log2(32 / NV) shuffles instead of
// 5 NV: in each step a lane hands one half of its values to its partner and keeps the other half.  On
// return v[0] of lane L is the total of value number L >> (5 - log2 NV).
template <int NV>
__device__ __forceinline__ void warp_multi_sum(float (&v)[NV], int lane) {
  static_assert(NV >= 2 && NV <= 32 && (NV & (NV - 1)) == 0, "a power of two");
  int off = 16;
#pragma unroll
  for (int cnt = NV; cnt > 1; cnt >>= 1, off >>= 1) {
    const int half = cnt >> 1;
    const bool upper = (lane & off) != 0;
#pragma unroll
    for (int k = 0; k < half; ++k) {
      const float send = upper ? v[k] : v[k + half];
      const float keep = upper ? v[k + half] : v[k];
      v[k] = keep + __shfl_xor_sync(0xffffffffu, send, off);
    }
  }
#pragma unroll
  for (; off > 0; off >>= 1) v[0] += __shfl_xor_sync(0xffffffffu, v[0], off);
}
__host__ __device__ constexpr int cl_pow2_at_least(int x) { return x <= 2 ? 2 : x <= 4 ? 4 : x <= 8 ? 8 : x <= 16 ? 16 : 32; }
__host__ __device__ constexpr int cl_log2(int x) { return x <= 2 ? 1 : x <= 4 ? 2 : x <= 8 ? 3 : x <= 16 ? 4 : 5; }

// Combines partial results (one per lane; lanes without one pass m = -3e38, S = 0, pos = INT_MAX) across
// the warp: the maximum, the lowest position among those that attain it, the sums rescaled to it.
template <typename T>
__device__ __forceinline__ void cl_warp_combine(float& m, int& pos, float& S, float& sum_z, float& S_T, bool temp, float inv_T) {
  const unsigned key = float_order_key(m + 0.f);
  const unsigned key_m = __reduce_max_sync(0xffffffffu, key);
  const float mm = float_from_order_key(key_m);
  pos = (int)__reduce_min_sync(0xffffffffu, key == key_m ? (unsigned)pos : 0x7fffffffu);
  S = warp_sum(S * rescale_exp2<T>((m - mm) * kLog2e));
  if (temp) S_T = warp_sum(S_T * rescale_exp2<T>((m - mm) * (kLog2e * inv_T)));
  sum_z = warp_sum(sum_z);
  m = mm;
}

// What pass B needs of the row statistics (registers), and its running sums.
template <int N, int NS>
struct ClColCtx {
  float nml[N], cpi[N];          // per model: -maximum * log2(e) (bf16 logits) or -maximum (fp32 logits), and w / S
  float cti[NS], lsi[NS];        // KL: 1 / S_T and log S_T (slot N: the averaged peers)
  float mb;                      // KL mean target: maximum of the averaged peers
  float cd, cq, cy, ckl, inv_T;
  bool t_one, centred;
  int y;
  const ClStat* stat;            // shared memory: the full statistics (maxima for the KL logarithms, class means)
  float cmean;                   // centred distance: average over the models of their class means
  float inv_C;
};
template <int NOUT>
struct ClColAcc {
  float2 dist2[NOUT], qs2;
};

// exp(z - m) for a pair of columns from the precomputed -m (see ClColCtx::nml)
template <typename T>
__device__ __forceinline__ float2 exp_from_nml(float2 z, float nml) {
  if constexpr (sizeof(T) == 4) {
    return make_float2(expf(z.x + nml), expf(z.y + nml));
  } else {
    const float2 t = __ffma2_rn(z, make_float2(kLog2e, kLog2e), make_float2(nml, nml));
    return make_float2(ex2_approx(t.x), ex2_approx(t.y));
  }
}

// Two neighbouring columns c, c + 1 of the n models (zc): distance terms into `acc`, gradient pairs of the
// requested models into gc.  LAB: c or c + 1 may be the label column.  MASKED: the distance terms of the two
// columns count with the weights in2 (1 / 0: a column outside the row, or a column done before, adds nothing).
template <typename T, int N, int MODE, bool ALL, bool LAB, bool MASKED, int NS>
__device__ __forceinline__ void cl_column2(const ClColCtx<N, NS>& x, ClColAcc<ALL ? N : 1>& acc, const float2 (&zc)[N],
                                           float2 (&gc)[ALL ? N : 1], int64_t c, float2 in2) {
  constexpr int NOUT = ALL ? N : 1;
  float2 ncq = make_float2(-x.cq, -x.cq);
  if constexpr (LAB) ncq = make_float2((c == (int64_t)x.y) ? -(x.cq + x.cy) : -x.cq, (c + 1 == (int64_t)x.y) ? -(x.cq + x.cy) : -x.cq);
  auto counted = [&](float2 v) { if constexpr (MASKED) return __fmul2_rn(v, in2); else return v; };
  if constexpr (MODE == kClMse) {
    // z'_i = z_i - mean_j z_j; for the centred distance z_i loses the class mean of model i first
    float2 zp[N], mu = zc[0];
#pragma unroll
    for (int i = 1; i < N; ++i) mu = __fadd2_rn(mu, zc[i]);
    mu = __fmul2_rn(mu, make_float2(-1.f / (float)N, -1.f / (float)N));
#pragma unroll
    for (int i = 0; i < N; ++i) zp[i] = __fadd2_rn(zc[i], mu);
    if (x.centred) {
#pragma unroll
      for (int i = 0; i < N; ++i) {
        const float d = x.cmean - x.stat[i].sum_z * x.inv_C;
        zp[i] = __fadd2_rn(zp[i], make_float2(d, d));
      }
    }
    if constexpr (!ALL) {   // sum_j z'_j^2 of the pairwise form (with every model's output it is the sum of their distance sums)
      float2 q = make_float2(0.f, 0.f);
#pragma unroll
      for (int i = 0; i < N; ++i) q = __ffma2_rn(zp[i], zp[i], q);
      acc.qs2 = __fadd2_rn(acc.qs2, counted(q));
    }
#pragma unroll
    for (int i = 0; i < NOUT; ++i) {
      const float2 e = exp_from_nml<T>(zc[i], x.nml[i]);
      gc[i] = __ffma2_rn(e, make_float2(x.cpi[i], x.cpi[i]), __ffma2_rn(make_float2(x.cd, x.cd), zp[i], ncq));
      acc.dist2[i] = __ffma2_rn(counted(zp[i]), zp[i], acc.dist2[i]);
    }
  } else if constexpr (MODE == kClKlPairwise) {
    float2 t[N], lt[N], Q = make_float2(0.f, 0.f), E = make_float2(0.f, 0.f);
#pragma unroll
    for (int i = 0; i < N; ++i) {
      const float mi = x.stat[i].m;
      float2 e1 = make_float2(0.f, 0.f);
      if (x.t_one || i < NOUT) e1 = exp_from_nml<T>(zc[i], x.nml[i]);
      const float2 et = x.t_one ? e1 : exp_temp2<T>(zc[i], mi, x.inv_T, kLog2e * x.inv_T);
      t[i] = __fmul2_rn(et, make_float2(x.cti[i], x.cti[i]));
      const float2 d = __fadd2_rn(zc[i], make_float2(-mi, -mi));
      const float2 l = __ffma2_rn(d, make_float2(x.inv_T, x.inv_T), make_float2(-x.lsi[i], -x.lsi[i]));
      lt[i] = make_float2(fmaxf(l.x, -3.0e38f), fmaxf(l.y, -3.0e38f));   // log t_i, kept finite: 0 * log 0 = 0
      Q = __fadd2_rn(Q, t[i]);
      E = __ffma2_rn(t[i], lt[i], E);
      if (i < NOUT) gc[i] = __ffma2_rn(e1, make_float2(x.cpi[i], x.cpi[i]), ncq);
    }
    const float2 nQ = make_float2(-Q.x, -Q.y);
#pragma unroll
    for (int i = 0; i < NOUT; ++i) {
      gc[i] = __ffma2_rn(make_float2(x.ckl, x.ckl), __ffma2_rn(make_float2((float)N, (float)N), t[i], nQ), gc[i]);
      acc.dist2[i] = __fadd2_rn(acc.dist2[i], counted(__ffma2_rn(nQ, lt[i], E)));   // sum_{j != i} t_j (log t_j - log t_i)
    }
  } else {
    // KL to the softmax of the averaged peers: t = softmax(zbar / T), p^T = softmax(z_0 / T)
    const float inv_P = 1.f / (float)(N - 1);
    const float m0 = x.stat[0].m;
    float2 zb = zc[1];
#pragma unroll
    for (int j = 2; j < N; ++j) zb = __fadd2_rn(zb, zc[j]);
    zb = __fmul2_rn(zb, make_float2(inv_P, inv_P));
    const float2 e1 = exp_from_nml<T>(zc[0], x.nml[0]);
    const float2 eT = x.t_one ? e1 : exp_temp2<T>(zc[0], m0, x.inv_T, kLog2e * x.inv_T);
    const float2 pT = __fmul2_rn(eT, make_float2(x.cti[0], x.cti[0]));
    const float2 x0 = __fadd2_rn(zc[0], make_float2(-m0, -m0));
    const float2 lp = __ffma2_rn(x0, make_float2(x.inv_T, x.inv_T), make_float2(-x.lsi[0], -x.lsi[0]));
    const float2 tb = __fmul2_rn(exp_temp2<T>(zb, x.mb, x.inv_T, kLog2e * x.inv_T), make_float2(x.cti[N], x.cti[N]));
    const float2 xb = __fadd2_rn(zb, make_float2(-x.mb, -x.mb));
    const float2 lb = __ffma2_rn(xb, make_float2(x.inv_T, x.inv_T), make_float2(-x.lsi[N], -x.lsi[N]));
    const float2 dl = make_float2(fmaxf(lb.x, -3.0e38f) - fmaxf(lp.x, -3.0e38f), fmaxf(lb.y, -3.0e38f) - fmaxf(lp.y, -3.0e38f));
    gc[0] = __ffma2_rn(make_float2(x.ckl, x.ckl), __fadd2_rn(pT, make_float2(-tb.x, -tb.y)),
                       __ffma2_rn(e1, make_float2(x.cpi[0], x.cpi[0]), ncq));
    acc.dist2[0] = __ffma2_rn(counted(tb), dl, acc.dist2[0]);
  }
}

// One segment off the fast path, element by element: a ragged segment (columns outside the row contribute nothing
// and are not written), or -- with `count` false -- the segment that holds the label column, whose gradient
// elements are written once more with the label's term (the fast path wrote them without it).
// (context and sums in and out by value, so that the caller's copies stay in registers)
template <typename T, int N, int MODE, bool ALL, int NS>
__device__ __noinline__ ClColAcc<ALL ? N : 1> cl_slow_segment(ClColCtx<N, NS> x, ClColAcc<ALL ? N : 1> acc, const char* slices, uint32_t slice_bytes,
                                                              int q, int64_t cbase, int64_t C, bool count, bool only_label, void* const* grad,
                                                              int64_t img_off, int s) {
  constexpr int H = SegOps<T>::H;
  constexpr int NOUT = ALL ? N : 1;
#pragma unroll 1
  for (int h = 0; h < H; ++h) {
    float2 zc[N], gc[NOUT];
    const int64_t c0 = cbase + 2 * h;
    const bool in0 = c0 >= 0 && c0 < C, in1 = c0 + 1 >= 0 && c0 + 1 < C;
    const bool st0 = in0 && (!only_label || c0 == (int64_t)x.y), st1 = in1 && (!only_label || c0 + 1 == (int64_t)x.y);
    if (!st0 && !st1 && !(count && (in0 || in1))) continue;
#pragma unroll
    for (int i = 0; i < N; ++i) {
      const T* el = reinterpret_cast<const T*>(slices + (size_t)i * slice_bytes + (size_t)q * 16) + 2 * h;
      const float mi = x.stat[i].m;
      zc[i] = make_float2(in0 ? Elem<T>::to_f32(el[0]) : mi, in1 ? Elem<T>::to_f32(el[1]) : mi);
    }
    cl_column2<T, N, MODE, ALL, true, true>(x, acc, zc, gc, c0, make_float2(count && in0 ? 1.f : 0.f, count && in1 ? 1.f : 0.f));
#pragma unroll
    for (int i = 0; i < NOUT; ++i) {
      if (grad[i] == nullptr) continue;
      T* ge = reinterpret_cast<T*>(reinterpret_cast<char*>(grad[i]) + img_off + (size_t)s * 16) + 2 * h;
      if (st0) ge[0] = Elem<T>::from_f32(gc[i].x);
      if (st1) ge[1] = Elem<T>::from_f32(gc[i].y);
    }
  }
  return acc;
}

// ------------------------------------------------------------------ the kernel
// T: element type; N: resident tensors; MODE: ClMode; ALL: every model's outputs (else model 0's only).
template <typename T, int N, int MODE, bool ALL>
__global__ void __launch_bounds__(kClThreads, 2) rows_cluster_kernel(const __grid_constant__ ClArgs a) {
  constexpr int V = SegOps<T>::V;
  constexpr int H = SegOps<T>::H;
  constexpr int ES = (int)sizeof(T);
  constexpr bool KL = MODE != kClMse;
  constexpr bool KLM = MODE == kClKlMeanTarget;
  constexpr int NOUT = ALL ? N : 1;
  constexpr int NSTAT = KLM ? N + 1 : N;
  constexpr int NS = KL ? NSTAT : 1;
  constexpr int NW = kClWarps, NT = kClThreads;
  static_assert(!(KLM && ALL), "the mean-target KL distance is a single-model form");
  static_assert(N >= 2 && N <= kClMax, "tensor count");
  extern __shared__ __align__(128) unsigned char smem_raw[];
  ClCtrl* ctrl = reinterpret_cast<ClCtrl*>(smem_raw);
  char* slices = reinterpret_cast<char*>(smem_raw) + kClCtrlBytes;
  cg::cluster_group cluster = cg::this_cluster();
  const int K = (int)cluster.num_blocks();
  const int rank = (int)cluster.block_rank();
  const int cid = (int)(blockIdx.x / K), ncl = (int)(gridDim.x / K);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t C = a.classes, R = a.rows_total;
  const float inv_C = 1.f / (float)C;
  const float inv_T = KL ? 1.f / a.temperature : 1.f;
  const bool t_one = !KL || a.temperature == 1.f;
  const bool need_z = a.eps != 0.f || a.centred != 0;   // sum_c z_c enters the smoothed task loss and the class means
  const bool want_grad = a.grad[0] != nullptr;

  if (tid == 0) {
    for (int i = 0; i < N; ++i) mbar_init(&ctrl->full[i], 1);
    ctrl->abort_flag = 0;
    mbar_init_fence();
  }
  wait_for_prior_grid();  // from here on the workspace header and the valid-row counts are read
  __syncthreads();

  float w = 1.f;
  if (a.reduction == CODISTILL_REDUCE_MEAN_VALID) {
    const int nb = a.hdr->prep_blocks;
    int64_t nv = 0;
    for (int b = 0; b < nb; ++b) nv += a.partials[2 * b];
    w = 1.f / (float)(nv > 1 ? nv : 1);
  }
  constexpr float kRatio = (float)N / (float)(N - 1);                 // z_i - zbar_(-i) = kRatio * z'_i
  ClColCtx<N, NS> cx;
  cx.cd = w * a.alpha * (2.f * inv_C) * kRatio;                        // z'_i -> w alpha dD_i/dz_i      (MSE)
  cx.cq = w * a.eps * inv_C;
  cx.cy = w * (1.f - a.eps);
  cx.ckl = KLM ? w * a.alpha * a.temperature                           // (p^T - t) -> w alpha dD/dz
               : w * a.alpha * a.temperature / (float)(N - 1);         // (n t_i - Q) -> w alpha dD_i/dz_i
  cx.inv_T = inv_T;
  cx.t_one = t_one;
  cx.centred = a.centred != 0;
  cx.mb = 0.f;
  cx.stat = ctrl->stat;
  cx.inv_C = inv_C;
  cx.cmean = 0.f;
  const int seg_begin = rank * a.spc;

  auto row_is_valid = [&](long long r) {
    if (a.mask != nullptr && a.mask[r] == 0) return false;
    const int32_t y = a.labels[r];
    return y >= 0 && (int64_t)y < C;
  };
  // Thread 0: start the bulk copies of this CTA's range of row r for all n tensors.
  auto issue_row = [&](long long r) {
    const int64_t lr = r - a.row_begin;
    const RowGeom g = row_geom<T>(lr, a.row_stride, C);
    const int seg_end = min(seg_begin + a.spc, g.n_seg);
    if (seg_end <= seg_begin) {
      for (int i = 0; i < N; ++i) mbar_arrive(&ctrl->full[i]);
      return;
    }
    const uint32_t begin = (uint32_t)seg_begin * 16u, end = (uint32_t)seg_end * 16u;
    // The last row of the whole call may end inside a segment that reaches past the tensor: that
    // segment is fetched element by element, whole-segment copies stop before it.
    const uint32_t valid_end = (uint32_t)(g.head + C) * ES;
    const bool clip = (r == R - 1) && ((a.row_stride - C) * ES < 16) && (valid_end & 15u) && end > (valid_end & ~15u);
    const uint32_t copy_end = clip ? (valid_end & ~15u) : end;
    const uint32_t bytes = copy_end > begin ? copy_end - begin : 0u;
    const int64_t img_off = (lr * a.row_stride - g.head) * ES;   // image start relative to the tensor
#pragma unroll 1
    for (int i = 0; i < N; ++i) {
      const char* src = reinterpret_cast<const char*>(a.model[i]) + img_off;
      char* dst = slices + (size_t)i * a.slice_bytes;
      if (clip) {
        for (uint32_t o = copy_end > begin ? copy_end : begin; o < valid_end; o += ES)
          *reinterpret_cast<T*>(dst + (o - begin)) = *reinterpret_cast<const T*>(src + o);
      }
      mbar_arrive_expect_tx(&ctrl->full[i], bytes);
      for (uint32_t o = 0; o < bytes; o += kClCopyPiece)
        bulk_g2s(dst + o, src + begin + o, bytes - o < kClCopyPiece ? bytes - o : kClCopyPiece, &ctrl->full[i]);
    }
  };
  // CTA 0: loss and flag word of the pending row with parity `pp`; every CTA has stored its distance
  // partial sums into this CTA's dgather before the cluster barrier that precedes this call.
  auto finish_row = [&](int pp) {
    for (int i = warp; i < NOUT; i += NW) {
      const float dsum = warp_sum(lane < K ? ctrl->dgather[pp][lane][i] : 0.f);
      const float qsum = warp_sum(lane < K ? ctrl->dgather[pp][lane][kClMax] : 0.f);
      if (lane == 0) {
        const ClStat st = ctrl->pend[pp][i];
        const long long r = ctrl->pend_row[pp];
        const int y = ctrl->pend_y[pp];
        const float ce = (st.m + logf(st.S)) - (1.f - a.eps) * st.zy - (a.eps * inv_C) * st.sum_z;
        float D;
        if constexpr (KLM) D = a.temperature * a.temperature * dsum;
        else if constexpr (KL) D = a.temperature * a.temperature * dsum / (float)(N - 1);
        else D = a.pairwise ? fmaf((float)N, dsum, qsum) * inv_C / (float)(N - 1) : dsum * kRatio * kRatio * inv_C;
        uint32_t flags = (st.col == y) ? 1u : 0u;
        int bit = 1;
        for (int j = 0; j < N; ++j) {
          if (j == i) continue;
          if (ctrl->pend[pp][j].col == st.col) flags |= (1u << bit);
          ++bit;
        }
        a.row_loss[(int64_t)i * R + r] = a.alpha != 0.f ? fmaf(a.alpha, D, ce) : ce;
        a.row_flags[(int64_t)i * R + r] = flags;
      }
    }
  };

  int v = 0;                   // valid rows done by this cluster
  long long issued = -1;       // thread 0: row whose copies were started last
  for (long long r = a.row_begin + cid; r < a.row_end; r += ncl) {
    const int64_t lr = r - a.row_begin;
    const RowGeom g = row_geom<T>(lr, a.row_stride, C);
    const int seg_end = min(seg_begin + a.spc, g.n_seg);
    const int nseg = seg_end > seg_begin ? seg_end - seg_begin : 0;     // segments of this CTA's range in this row
    // of which [q_lo, q_hi) are whole segments inside the row; a ragged first / last segment of the row image is
    // done apart by one thread (tid 0 / tid 32)
    const int q_lo = (seg_begin < g.seg_lo && nseg > 0) ? g.seg_lo - seg_begin : 0;
    const int q_hi = seg_end > g.seg_hi ? (g.seg_hi > seg_begin ? g.seg_hi - seg_begin : 0) : nseg;
    const bool edge_head = tid == 0 && q_lo > 0;
    const bool edge_tail = tid == 32 && q_hi < nseg && q_hi >= q_lo;
    const int q_edge = edge_head ? 0 : nseg - 1;
    const int64_t img_off = (lr * a.row_stride - g.head) * ES;
    const int y = a.labels[r];
    const bool valid = (a.mask == nullptr || a.mask[r] != 0) && y >= 0 && (int64_t)y < C;

    if (!valid) {  // masked row: zero gradient rows, no loss, no counts; nothing is read
      if (want_grad) {
#pragma unroll 1
        for (int i = 0; i < NOUT; ++i) {
          char* g_img = reinterpret_cast<char*>(a.grad[i]) + img_off;
          for (int q = q_lo + tid; q < q_hi; q += NT) *reinterpret_cast<uint4*>(g_img + (size_t)(seg_begin + q) * 16) = make_uint4(0u, 0u, 0u, 0u);
          if (edge_head || edge_tail) {
            const int s = seg_begin + q_edge;
#pragma unroll
            for (int e = 0; e < V; ++e) {
              const int64_t c = (int64_t)s * V - g.head + e;
              if (c >= 0 && c < C) reinterpret_cast<T*>(g_img + (size_t)s * 16)[e] = Elem<T>::from_f32(0.f);
            }
          }
        }
      }
      if (rank == 0 && tid < NOUT) { a.row_loss[(int64_t)tid * R + r] = 0.f; a.row_flags[(int64_t)tid * R + r] = 0u; }
      continue;
    }
    const int par = v & 1;
    if (tid == 0 && issued != r) { issue_row(r); issued = r; }

    // ================= pass A: statistics of this CTA's range, tensor by tensor as the copies land
    // Every warp takes a share of each tensor, so the sweep of tensor i runs while tensors i+1.. are still
    // in flight.  One lane per warp watches the copy barrier (with back-off): waiting warps take next to no
    // issue slots from the CTA that shares the SM.
    {
      ClLane L[N];
#pragma unroll
      for (int i = 0; i < N; ++i) {
        if (lane == 0) cl_wait(&ctrl->full[i], (uint32_t)v & 1u, ctrl, a.hdr);
        __syncwarp();
        const char* sl = slices + (size_t)i * a.slice_bytes;
        L[i] = t_one ? cl_sweep_range<T, false>(sl, q_lo, q_hi, seg_begin, tid, inv_T, need_z)
                     : cl_sweep_range<T, KL>(sl, q_lo, q_hi, seg_begin, tid, inv_T, need_z);
        if (edge_head || edge_tail) {
          const uint4 raw = *reinterpret_cast<const uint4*>(sl + (size_t)q_edge * 16);
          L[i] = t_one ? cl_sweep_edge<T, false>(L[i], raw, seg_begin + q_edge, g.head, C, inv_T)
                       : cl_sweep_edge<T, KL>(L[i], raw, seg_begin + q_edge, g.head, C, inv_T);
        }
      }
      // per tensor the warp's maximum and its first segment by integer reductions; then all the sums at once
      constexpr int NQ = KL ? 3 : 2;
      constexpr int NV = cl_pow2_at_least(NQ * N);
      float vals[NV];
#pragma unroll
      for (int k = 0; k < NV; ++k) vals[k] = 0.f;
#pragma unroll
      for (int i = 0; i < N; ++i) {
        const unsigned key = float_order_key(L[i].best + 0.f);   // -0 is folded onto +0: they tie
        const unsigned key_w = __reduce_max_sync(0xffffffffu, key);
        const int seg_w = (int)__reduce_min_sync(0xffffffffu, key == key_w ? (unsigned)L[i].seg : 0x7fffffffu);
        const float m_w = float_from_order_key(key_w);
        vals[i] = L[i].s * rescale_exp2<T>((L[i].best - m_w) * kLog2e);
        vals[N + i] = L[i].z;
        if constexpr (KL) vals[2 * N + i] = t_one ? 0.f : L[i].t * rescale_exp2<T>((L[i].best - m_w) * (kLog2e * inv_T));
        if (lane == 0) { ctrl->rec[warp][i].m = m_w; ctrl->rec[warp][i].seg = seg_w; }
      }
      warp_multi_sum<NV>(vals, lane);
      constexpr int kShift = 5 - cl_log2(NV);
      if ((lane & ((1 << kShift) - 1)) == 0) {
        const int j = lane >> kShift;
        if (j < NQ * N) {
          const int quantity = j / N, i = j - quantity * N;
          if (quantity == 0) ctrl->rec[warp][i].S = vals[0];
          else if (quantity == 1) ctrl->rec[warp][i].sum_z = vals[0];
          else ctrl->rec[warp][i].S_T = vals[0];
        }
      }
    }
    if constexpr (KLM) {
      // statistics of the averaged peer logits zbar = mean_{j >= 1} z_j at temperature T
      ClLane L;
      L.best = -3.0e38f; L.seg = 0x7fffffff; L.s = 0.f; L.z = 0.f; L.t = 0.f;
      const float inv_P = 1.f / (float)(N - 1);
      for (int q = tid; q < nseg; q += NT) {
        const int s = seg_begin + q;
        float2 zb[H];
#pragma unroll
        for (int h = 0; h < H; ++h) zb[h] = make_float2(0.f, 0.f);
#pragma unroll
        for (int j = 1; j < N; ++j) {
          float2 v2[H];
          SegOps<T>::unpack2(*reinterpret_cast<const uint4*>(slices + (size_t)j * a.slice_bytes + (size_t)q * 16), v2);
#pragma unroll
          for (int h = 0; h < H; ++h) zb[h] = __fadd2_rn(zb[h], v2[h]);
        }
        float fm = -3.0e38f;
        bool in[V];
#pragma unroll
        for (int e = 0; e < V; ++e) {
          const int64_t c = (int64_t)s * V - g.head + e;
          in[e] = c >= 0 && c < C;
        }
#pragma unroll
        for (int h = 0; h < H; ++h) {
          zb[h] = __fmul2_rn(zb[h], make_float2(inv_P, inv_P));
          if (in[2 * h]) fm = fmaxf(fm, zb[h].x);
          if (in[2 * h + 1]) fm = fmaxf(fm, zb[h].y);
        }
        const float nb = fmaxf(L.best, fm);
        L.t *= rescale_exp2<T>((L.best - nb) * (kLog2e * inv_T));
        L.best = nb;
#pragma unroll
        for (int h = 0; h < H; ++h) {
          const float2 e2 = exp_temp2<T>(zb[h], nb, inv_T, kLog2e * inv_T);
          if (in[2 * h]) L.t += e2.x;
          if (in[2 * h + 1]) L.t += e2.y;
        }
      }
      const float m_w = warp_max_redux(L.best);
      const float t_w = warp_sum(L.t * rescale_exp2<T>((L.best - m_w) * (kLog2e * inv_T)));
      if (lane == 0) { ClRec rc; rc.m = m_w; rc.seg = 0x7fffffff; rc.S = 0.f; rc.sum_z = 0.f; rc.S_T = t_w; rc.tensor = N; ctrl->rec[warp][N] = rc; }
    }
    __syncthreads();
    // This CTA's partial result of tensor i, by warp i: one warp's record per lane (the first segment that attains
    // the maximum is the lowest one among the records that attain it), handed to every CTA of the cluster.
    for (int i = warp; i < NSTAT; i += NW) {
      float m = -3.0e38f, S = 0.f, sum_z = 0.f, S_T = 0.f;
      int seg = 0x7fffffff;
      if (lane < NW) {
        const ClRec rc = ctrl->rec[lane][i];
        m = rc.m; S = rc.S; sum_z = rc.sum_z; S_T = rc.S_T; seg = rc.seg;
      }
      cl_warp_combine<T>(m, seg, S, sum_z, S_T, !t_one || i == N, inv_T);
      ClPart p;
      p.m = m; p.S = S; p.sum_z = sum_z; p.S_T = S_T; p.col = 0x7fffffff; p.zy = 0.f;
      if (i < N) {
        const T* sl = reinterpret_cast<const T*>(slices + (size_t)i * a.slice_bytes);
        if (seg >= seg_begin && seg < seg_end) {   // first column of that segment that attains the maximum
#pragma unroll
          for (int e = V - 1; e >= 0; --e) {
            const int64_t c = (int64_t)seg * V - g.head + e;
            if (c >= 0 && c < C && Elem<T>::to_f32(sl[(size_t)(seg - seg_begin) * V + e]) == m) p.col = (int)c;
          }
        }
        const int seg_y = (g.head + y) / V;
        if (seg_y >= seg_begin && seg_y < seg_end) p.zy = Elem<T>::to_f32(sl[(size_t)(seg_y - seg_begin) * V + (g.head + y) % V]);
      }
      if (lane < K) *cluster.map_shared_rank(&ctrl->gather[par][rank][i], lane) = p;
    }
    cluster.sync();   // every CTA's partial results of this row have arrived (and its work on the previous row is done)

    // ================= statistics of the whole row: warp i combines the K partial results of tensor i
    for (int i = warp; i < NSTAT; i += NW) {
      ClPart p;
      p.m = -3.0e38f; p.col = 0x7fffffff; p.S = 0.f; p.sum_z = 0.f; p.S_T = 0.f; p.zy = 0.f;
      if (lane < K) p = ctrl->gather[par][lane][i];
      ClStat st;
      st.m = p.m; st.col = p.col; st.S = p.S; st.sum_z = p.sum_z; st.S_T = p.S_T;
      cl_warp_combine<T>(st.m, st.col, st.S, st.sum_z, st.S_T, !t_one || i == N, inv_T);
      if (t_one && i < N) st.S_T = st.S;
      st.zy = warp_sum(p.zy);
      if (lane == 0) ctrl->stat[i] = st;
    }
    if (rank == 0 && v >= 1) finish_row(par ^ 1);   // the previous valid row: all its distance partials are in
    __syncthreads();
    if (rank == 0 && tid < NSTAT) {
      ctrl->pend[par][tid] = ctrl->stat[tid];
      if (tid == 0) { ctrl->pend_row[par] = r; ctrl->pend_y[par] = y; }
    }
    {
      float cm = 0.f;
#pragma unroll
      for (int i = 0; i < N; ++i) {
        const ClStat st = ctrl->stat[i];
        cx.nml[i] = ES == 4 ? -st.m : -st.m * kLog2e;
        cx.cpi[i] = w * __frcp_rn(st.S);
        cm += st.sum_z;
        if constexpr (KL) { cx.cti[i] = __frcp_rn(st.S_T); cx.lsi[i] = logf(st.S_T); }
      }
      cx.cmean = cm * inv_C / (float)N;
    }
    if constexpr (KLM) { const ClStat st = ctrl->stat[N]; cx.mb = st.m; cx.cti[N] = __frcp_rn(st.S_T); cx.lsi[N] = logf(st.S_T); }
    cx.y = y;

    // ================= pass B: distance terms and gradients, the n models side by side
    ClColAcc<NOUT> acc;
    acc.qs2 = make_float2(0.f, 0.f);
#pragma unroll
    for (int i = 0; i < NOUT; ++i) acc.dist2[i] = make_float2(0.f, 0.f);
#pragma unroll 1
    for (int q = q_lo + tid; q < q_hi; q += NT) {
      const int s = seg_begin + q;
      const int64_t cbase = (int64_t)s * V - g.head;
      uint4 rw[N];
#pragma unroll
      for (int i = 0; i < N; ++i) rw[i] = *reinterpret_cast<const uint4*>(slices + (size_t)i * a.slice_bytes + (size_t)q * 16);
#pragma unroll
      for (int h = 0; h < H; ++h) {
        float2 zc[N], gc[NOUT];
#pragma unroll
        for (int i = 0; i < N; ++i) {
          if constexpr (ES == 4) {
            zc[i] = h == 0 ? make_float2(__uint_as_float(rw[i].x), __uint_as_float(rw[i].y))
                           : make_float2(__uint_as_float(rw[i].z), __uint_as_float(rw[i].w));
          } else {
            const uint32_t word = h == 0 ? rw[i].x : h == 1 ? rw[i].y : h == 2 ? rw[i].z : rw[i].w;
            zc[i] = make_float2(__uint_as_float(word << 16), __uint_as_float(word & 0xFFFF0000u));
          }
        }
        cl_column2<T, N, MODE, ALL, false, false>(cx, acc, zc, gc, cbase + 2 * h, make_float2(1.f, 1.f));
#pragma unroll
        for (int i = 0; i < NOUT; ++i) {
          if constexpr (ES == 4) {
            if (h == 0) { rw[i].x = __float_as_uint(gc[i].x); rw[i].y = __float_as_uint(gc[i].y); }
            else { rw[i].z = __float_as_uint(gc[i].x); rw[i].w = __float_as_uint(gc[i].y); }
          } else {
            const __nv_bfloat162 pk = __floats2bfloat162_rn(gc[i].x, gc[i].y);
            const uint32_t word = *reinterpret_cast<const uint32_t*>(&pk);
            if (h == 0) rw[i].x = word; else if (h == 1) rw[i].y = word; else if (h == 2) rw[i].z = word; else rw[i].w = word;
          }
        }
      }
      if (want_grad) {
#pragma unroll
        for (int i = 0; i < NOUT; ++i) *reinterpret_cast<uint4*>(reinterpret_cast<char*>(a.grad[i]) + img_off + (size_t)s * 16) = rw[i];
      }
    }
    // the ragged segments, element by element
    if (edge_head || edge_tail)
      acc = cl_slow_segment<T, N, MODE, ALL>(cx, acc, slices, a.slice_bytes, q_edge, (int64_t)(seg_begin + q_edge) * V - g.head, C, true, false,
                                       a.grad, img_off, seg_begin + q_edge);
    // the label column: its gradient elements once more, now with the label's term (a label inside a ragged segment
    // has had it already).  The thread that wrote the segment above writes it again: its stores stay in order.
    {
      const int seg_y = (g.head + y) / V;
      const int qy = seg_y - seg_begin;
      if (want_grad && qy >= q_lo && qy < q_hi && (qy - q_lo) % NT == tid)
        acc = cl_slow_segment<T, N, MODE, ALL>(cx, acc, slices, a.slice_bytes, qy, (int64_t)seg_y * V - g.head, C, false, true, a.grad, img_off, seg_y);
    }

    // ================= distance partial sums of this CTA, handed to CTA 0 (which reads them behind the next cluster barrier)
    {
      constexpr int ND = cl_pow2_at_least(NOUT + 1);
      float dv[ND];
#pragma unroll
      for (int k = 0; k < ND; ++k) dv[k] = 0.f;
      float qt = acc.qs2.x + acc.qs2.y;
#pragma unroll
      for (int i = 0; i < NOUT; ++i) {
        dv[i] = acc.dist2[i].x + acc.dist2[i].y;
        if constexpr (ALL) qt += dv[i];
      }
      dv[NOUT] = MODE == kClMse ? qt : 0.f;
      warp_multi_sum<ND>(dv, lane);
      constexpr int kShiftD = 5 - cl_log2(ND);
      if ((lane & ((1 << kShiftD) - 1)) == 0) {
        const int j = lane >> kShiftD;
        if (j <= NOUT) ctrl->dwarp[warp][j == NOUT ? kClMax : j] = dv[0];
      }
    }
    __syncthreads();   // pass B has read the ranges: they may be overwritten; the warps' partial sums are in place
    if (tid == 0) {
      // start the copies of the next valid row of this cluster behind the arithmetic of other CTAs on this SM
      long long r2 = r + ncl;
      while (r2 < a.row_end && !row_is_valid(r2)) r2 += ncl;
      if (r2 < a.row_end) { issue_row(r2); issued = r2; }
    }
    if (tid >= 32 && tid - 32 <= kClMax && (tid - 32 < NOUT || tid - 32 == kClMax)) {
      const int i = tid - 32;
      float d = 0.f;
#pragma unroll
      for (int wv = 0; wv < NW; ++wv) d += ctrl->dwarp[wv][i];
      *cluster.map_shared_rank(&ctrl->dgather[par][rank][i], 0) = d;
    }
    ++v;
  }

  // ---------------- the last valid row's loss; nobody leaves while its shared memory may still be written
  cluster.sync();
  if (rank == 0 && v >= 1) finish_row((v - 1) & 1);
  if (ctrl->abort_flag && tid == 0) {
    // a wait ran out: give copies that may still be in flight one more bounded interval before the CTA ends
    for (int i = 0; i < N; ++i)
      mbar_wait_limited(&ctrl->full[i], (uint32_t)(v + 1) & 1u, &ctrl->abort_flag, &a.hdr->status, CODISTILL_DEV_TIMEOUT, kClDrainLimitNs, false, true);
  }
}

// ------------------------------------------------------------------ host side
struct ClPlan {
  int cluster;           // CTAs per cluster (0: the kernel does not take the call)
  int spc;
  uint32_t slice_bytes;
  uint32_t smem_bytes;
};

static int cluster_size_override() {
  const char* s = getenv("CODISTILL_CLUSTER_SIZE");
  if (s == nullptr) return 0;
  const int k = atoi(s);
  return (k == 1 || k == 2 || k == 4 || k == 8 || k == 16) ? k : 0;
}

// Smallest cluster whose CTAs keep their share of the n row images in about half an SM's shared
// memory (two CTAs per SM: one computes while the other's copies are in flight).
ClPlan cluster_plan(int n, int64_t classes, int64_t row_stride, int dtype, int smem_optin) {
  ClPlan p = {0, 0, 0, 0};
  if (n < 2 || n > kClMax) return p;
  const int64_t n_seg = dtype == CODISTILL_F32 ? max_row_segments<float>(row_stride, classes)
                                               : max_row_segments<__nv_bfloat16>(row_stride, classes);
  if (n_seg * 16 < 8192 || classes > (int64_t)1 << 24) return p;
  const int64_t half = ((int64_t)smem_optin + 1024) / 2 - 1024;
  const int forced = cluster_size_override();
  for (int k = forced ? forced : 1; k <= (forced ? forced : kClMaxCluster); k *= 2) {
    const int64_t spc = (n_seg + k - 1) / k;
    const int64_t slice = (spc * 16 + 127) & ~(int64_t)127;
    const int64_t smem = kClCtrlBytes + (int64_t)n * slice;
    if (smem <= (forced ? (int64_t)smem_optin : half)) {
      p.cluster = k;
      p.spc = (int)spc;
      p.slice_bytes = (uint32_t)slice;
      p.smem_bytes = (uint32_t)smem;
      return p;
    }
  }
  return p;
}

template <typename T, int N, int MODE, bool ALL>
static cudaError_t cluster_launch_one(const ClArgs& a, const ClPlan& p, cudaStream_t stream) {
  auto kernel = rows_cluster_kernel<T, N, MODE, ALL>;
  // per kernel: the number of co-resident clusters of a launch shape is asked once per device, and the
  // kernel's shared-memory limit is only ever raised (a lower value would refuse earlier, larger shapes)
  static std::mutex mu;
  static std::map<std::tuple<int, int, uint32_t>, int> known;
  static std::map<int, uint32_t> smem_limit;
  int dev = 0;
  cudaError_t e = cuda_note(cudaGetDevice(&dev), "cudaGetDevice");
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(kClThreads);
  cfg.dynamicSmemBytes = p.smem_bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)p.cluster;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int max_clusters = 0;
  {
    std::lock_guard<std::mutex> lock(mu);
    const auto key = std::make_tuple(dev, p.cluster, p.smem_bytes);
    const auto it = known.find(key);
    if (it != known.end()) {
      max_clusters = it->second;
    } else {
      if (p.smem_bytes > smem_limit[dev]) {
        if ((e = cuda_note(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem_bytes),
                           "cudaFuncSetAttribute (shared memory size, cluster kernel)")) != cudaSuccess) return e;
        smem_limit[dev] = p.smem_bytes;
      }
      if (p.cluster > 8 && (e = cuda_note(cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1), "cudaFuncSetAttribute (cluster size)")) != cudaSuccess) return e;
      cfg.gridDim = dim3((unsigned)p.cluster);
      if ((e = cuda_note(cudaOccupancyMaxActiveClusters(&max_clusters, kernel, &cfg), "cudaOccupancyMaxActiveClusters")) != cudaSuccess) return e;
      if (max_clusters < 1) return cuda_note(cudaErrorLaunchOutOfResources, "no cluster of this size fits the device");
      known[key] = max_clusters;
      if (getenv("CODISTILL_VERBOSE"))
        fprintf(stderr, "codistill: cluster kernel n=%d: %d CTAs per cluster, %u bytes of shared memory per CTA, %d clusters co-resident\n",
                N, p.cluster, p.smem_bytes, max_clusters);
    }
  }
  const int64_t rows = a.row_end - a.row_begin;
  const int64_t clusters = rows < max_clusters ? rows : max_clusters;
  cfg.gridDim = dim3((unsigned)(clusters * p.cluster));
  cfg.numAttrs = 2;
  e = cuda_note(cudaLaunchKernelEx(&cfg, kernel, a), "cudaLaunchKernelEx (cluster kernel)");
  return e != cudaSuccess ? e : cudaGetLastError();
}

template <typename T, int N>
static cudaError_t cluster_launch_n(const ClArgs& a, const ClPlan& p, int mode, bool all, cudaStream_t stream) {
  if (mode == kClMse) return all ? cluster_launch_one<T, N, kClMse, true>(a, p, stream) : cluster_launch_one<T, N, kClMse, false>(a, p, stream);
  if (mode == kClKlPairwise)
    return all ? cluster_launch_one<T, N, kClKlPairwise, true>(a, p, stream) : cluster_launch_one<T, N, kClKlPairwise, false>(a, p, stream);
  return all ? cudaErrorNotSupported : cluster_launch_one<T, N, kClKlMeanTarget, false>(a, p, stream);
}

template <typename T>
static cudaError_t cluster_launch_t(const ClArgs& a, const ClPlan& p, int mode, bool all, cudaStream_t stream) {
  switch (a.n) {
    case 2: return cluster_launch_n<T, 2>(a, p, mode, all, stream);
    case 3: return cluster_launch_n<T, 3>(a, p, mode, all, stream);
    case 4: return cluster_launch_n<T, 4>(a, p, mode, all, stream);
    case 5: return cluster_launch_n<T, 5>(a, p, mode, all, stream);
    case 6: return cluster_launch_n<T, 6>(a, p, mode, all, stream);
    case 7: return cluster_launch_n<T, 7>(a, p, mode, all, stream);
    case 8: return cluster_launch_n<T, 8>(a, p, mode, all, stream);
    default: return cudaErrorNotSupported;
  }
}

// Launches the cluster-resident kernel for rows [row_begin, row_end).  `mode`: ClMode; `all`: every model's outputs.
cudaError_t launch_cluster(ClArgs a, int dtype, int mode, bool all, int smem_optin, cudaStream_t stream) {
  const ClPlan p = cluster_plan(a.n, a.classes, a.row_stride, dtype, smem_optin);
  if (p.cluster == 0) return cudaErrorNotSupported;
  if (a.row_end <= a.row_begin) return cudaSuccess;
  a.spc = p.spc;
  a.slice_bytes = p.slice_bytes;
  return dtype == CODISTILL_F32 ? cluster_launch_t<float>(a, p, mode, all, stream) : cluster_launch_t<__nv_bfloat16>(a, p, mode, all, stream);
}

bool cluster_fits(int n, int64_t classes, int64_t row_stride, int dtype, int smem_optin) {
  return cluster_plan(n, classes, row_stride, dtype, smem_optin).cluster != 0;
}

// Whether the single-model call described by `a` can be served by the cluster-resident kernel.
bool cluster_supported(const KArgs& a, int dtype, int smem_optin) {
  if (a.n_peers < 1 || a.n_peers + 1 > kClMax) return false;
  if (a.dist != CODISTILL_DIST_MSE_LOGITS && a.dist != CODISTILL_DIST_KL_SOFTMAX && a.dist != CODISTILL_DIST_MSE_CENTRED) return false;
  uintptr_t bits = reinterpret_cast<uintptr_t>(a.own) | reinterpret_cast<uintptr_t>(a.grad);
  for (int j = 0; j < a.n_peers; ++j) bits |= reinterpret_cast<uintptr_t>(a.peers[j]);
  if (bits & 15u) return false;
  return cluster_plan(a.n_peers + 1, a.classes, a.row_stride, dtype, smem_optin).cluster != 0;
}

// The single-model call on the cluster-resident kernel: own logits as model 0, the peers behind it.
cudaError_t launch_cluster_single(const KArgs& k, int dtype, int smem_optin, cudaStream_t stream) {
  ClArgs a;
  memset(&a, 0, sizeof(a));
  a.model[0] = k.own;
  for (int j = 0; j < k.n_peers; ++j) a.model[1 + j] = k.peers[j];
  a.grad[0] = k.grad;
  a.labels = k.labels;
  a.mask = k.mask;
  a.row_loss = k.row_loss;
  a.row_flags = k.row_flags;
  a.hdr = k.hdr;
  a.partials = k.partials;
  a.rows_total = k.rows_total;
  a.row_begin = k.row_begin;
  a.row_end = k.row_end;
  a.classes = k.classes;
  a.row_stride = k.row_stride;
  a.n = k.n_peers + 1;
  a.pairwise = k.peer_reduce == CODISTILL_PEERS_PAIRWISE_MEAN;
  a.reduction = k.reduction;
  a.centred = k.dist == CODISTILL_DIST_MSE_CENTRED;
  a.alpha = k.alpha;
  a.eps = k.eps;
  a.temperature = k.temperature;
  int mode = kClMse;
  if (k.dist == CODISTILL_DIST_KL_SOFTMAX)
    mode = (k.peer_reduce == CODISTILL_PEERS_PAIRWISE_MEAN || k.n_peers == 1) ? kClKlPairwise : kClKlMeanTarget;
  return launch_cluster(a, dtype, mode, false, smem_optin, stream);
}

}  // namespace codistill
