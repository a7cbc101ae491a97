/*
 * codistill_oracle.c -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, double-precision CPU statement of the codistillation objective and of its
 * gradient with respect to the own logits.  It exists so that the CUDA library can be checked
 * against something that can be compared with the paper by eye.  Only the tests, the smoke
 * check and the benchmark's CPU-baseline leg may call it; it shares no code with the CUDA path.
 *
 * What it follows (arXiv 2010.02838, "A Closer Look at Codistillation for Distributed Training"):
 *   - Algorithm 1, the update of model i: the objective is
 *         L(y, f_i(x)) + alpha * 1/(n-1) * sum_{j != i} D(f_i(x), f_j(x)),
 *     differentiated with respect to model i only (peers are constants; Section 3).
 *   - Section 2: L is a standard supervised loss, cross-entropy here; earlier work used the
 *     KL divergence for D with alpha = 1.
 *   - Appendix "Implementation Details": D is the mean squared error between the logits of
 *     the two models, not centred; the same passage says that centring the logits gave similar
 *     results: the centred variant (each model's logits minus their mean over the classes before the
 *     squared error, i.e. the variance over the classes of the difference) is dist_kind 2.
 *   - Section 2 does not fix the direction of the KL divergence; the peer-as-target direction is dist_kind 1,
 *     the other direction dist_kind 3 and their average dist_kind 4.
 *   - Section 3 / Section 5: the term may be omitted (non-communication steps), n = 1 is
 *     ordinary training.
 * Readings where the paper is silent: label smoothing is uniform, q = (1 - eps) onehot(y) + eps / C;
 * a padding mask is one byte per row (non-zero = valid), masked rows give zero loss and gradient;
 * the KL form is T^2 KL(softmax(peer / T) || softmax(own / T)) with the peer as target; the reduced
 * loss is the mean over valid rows (or the sum) and the gradient is the gradient of that; the first
 * (lowest) index wins arg-max ties and -0.0 ties with +0.0.
 *
 * Pins: every function here is pinned by tests/test_oracle_pins.py (closed forms, a hand
 * example, invariants, finite differences, a float64 autograd composition of library ops,
 * brute force for the counters).  Nothing is "parity unpinned".
 *
 * Parallelism: rows only (OpenMP); the arithmetic of one row is strictly sequential in the
 * order written below.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_F32 = 0, ORACLE_BF16 = 1 };
enum { ORACLE_DIST_MSE = 0, ORACLE_DIST_KL = 1, ORACLE_DIST_MSE_CENTRED = 2,
       ORACLE_DIST_KL_REVERSE = 3,   /* T^2 KL(softmax(own / T) || softmax(peer / T)): the other direction of Section 2's KL */
       ORACLE_DIST_KL_SYMMETRIC = 4  /* half the sum of the two directions */ };
enum { ORACLE_PEERS_PAIRWISE = 0, ORACLE_PEERS_MEAN_TARGET = 1 };
enum { ORACLE_REDUCE_MEAN_VALID = 0, ORACLE_REDUCE_SUM = 1 };
enum { ORACLE_STATUS_BAD_LABEL = 1 };

/* Exact widening of one stored element to double. bf16 is the upper half of an IEEE binary32. */
static double load_elem(const void* base, int dtype, int64_t index) {
  if (dtype == ORACLE_F32) return (double)((const float*)base)[index];
  uint32_t bits = ((uint32_t)((const uint16_t*)base)[index]) << 16;
  float f;
  memcpy(&f, &bits, sizeof f);
  return (double)f;
}

/* log(sum_c exp(v_c)) by the max-shifted form; also returns the first index of the maximum. */
static double log_sum_exp(const double* v, int64_t C, int64_t* argmax_out) {
  double m = v[0];
  int64_t a = 0;
  for (int64_t c = 1; c < C; ++c)
    if (v[c] > m) { m = v[c]; a = c; } /* strict '>' : lowest index wins ties, -0.0 == +0.0 */
  double s = 0.0;
  for (int64_t c = 0; c < C; ++c) s += exp(v[c] - m);
  if (argmax_out) *argmax_out = a;
  return m + log(s);
}

/*
 * The softmax-KL family between own logits z and target logits v (a peer, or the mean of the peers), both
 * at temperature T, with p = softmax(z / T), t = softmax(v / T):
 *   forward  T^2 KL(t || p) = T^2 sum_c t_c (log t_c - log p_c),   d/dz_k = T (p_k - t_k)
 *   reverse  T^2 KL(p || t) = T^2 sum_c p_c (log p_c - log t_c),   d/dz_k = T p_k ((log p_k - log t_k) - KL(p || t))
 * weighted by wf and wr (1, 0: forward; 0, 1: reverse; 1/2, 1/2: symmetric).  Returns the weighted value and adds
 * scale times its derivative to dD.  lse_z = log sum exp(z / T); tmp is scratch of C doubles.
 */
static double kl_family(const double* z, const double* v, int64_t C, double T, double lse_z, double wf, double wr,
                        double scale, double* dD, double* tmp) {
  for (int64_t c = 0; c < C; ++c) tmp[c] = v[c] / T;
  const double lse_v = log_sum_exp(tmp, C, NULL);
  double kl_f = 0.0, kl_r = 0.0;
  for (int64_t c = 0; c < C; ++c) {
    const double log_t = v[c] / T - lse_v;
    const double log_p = z[c] / T - lse_z;
    kl_f += exp(log_t) * (log_t - log_p);
    kl_r += exp(log_p) * (log_p - log_t);
  }
  for (int64_t c = 0; c < C; ++c) {
    const double log_t = v[c] / T - lse_v;
    const double log_p = z[c] / T - lse_z;
    const double p = exp(log_p), t = exp(log_t);
    dD[c] += scale * (wf * T * (p - t) + wr * T * p * ((log_p - log_t) - kl_r));
  }
  return T * T * (wf * kl_f + wr * kl_r);
}

/* A row takes part iff its mask byte is non-zero (or there is no mask) and its label is a class id. */
static int row_is_valid(const int32_t* labels, const uint8_t* mask, int64_t r, int64_t C, int* bad_label) {
  if (mask && mask[r] == 0) return 0;
  if (labels[r] < 0 || (int64_t)labels[r] >= C) { *bad_label = 1; return 0; }
  return 1;
}

int codistill_oracle_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/*
 * own, peers[j]     [rows, row_stride] in `dtype`; peers has n-1 entries (ignored when n == 1)
 * grad_begin/end    rows for which the gradient is written: grad is [(grad_end-grad_begin), classes] doubles
 *                   (dense); pass grad = NULL to skip the gradient.
 * row_loss          [rows] doubles or NULL; reduced_loss [1]; counters [3 + (n-1)] int64 or NULL; status [1] or NULL
 * nthreads          OpenMP threads over rows (<= 0: library default)
 * returns 0, or 1 on invalid arguments.
 */
int codistill_oracle(const void* own, const void* const* peers, const int32_t* labels, const uint8_t* mask,
                     int n, int64_t rows, int64_t classes, int64_t row_stride, int dtype, double alpha,
                     double temperature, double label_smoothing, int dist_kind, int peer_reduce, int reduction,
                     int64_t grad_begin, int64_t grad_end, double* row_loss, double* reduced_loss, double* grad,
                     int64_t* counters, int32_t* status, int nthreads) {
  if (n < 1 || rows < 0 || classes < 1 || row_stride < classes || temperature <= 0.0) return 1;
  if (dtype != ORACLE_F32 && dtype != ORACLE_BF16) return 1;
  if (label_smoothing < 0.0 || label_smoothing >= 1.0) return 1;
  if (grad && (grad_begin < 0 || grad_end > rows || grad_begin > grad_end)) return 1;

  const int64_t C = classes;
  const int P = n - 1;                              /* number of peers */
  const int with_term = (P >= 1 && alpha != 0.0);   /* Section 3: the term may be absent; n = 1 is plain training */
  const double T = temperature, eps = label_smoothing;

  /* valid / masked rows first: the MEAN_VALID weight needs n_valid before any gradient */
  int64_t n_valid = 0, n_masked = 0;
  int any_bad = 0;
  for (int64_t r = 0; r < rows; ++r) {
    int bad = 0;
    if (row_is_valid(labels, mask, r, C, &bad)) ++n_valid; else ++n_masked;
    any_bad |= bad;
  }
  const double w = (reduction == ORACLE_REDUCE_SUM) ? 1.0 : 1.0 / (double)(n_valid > 1 ? n_valid : 1);

  double* loss_rows = (double*)calloc((size_t)(rows > 0 ? rows : 1), sizeof(double));
  int64_t* correct_rows = (int64_t*)calloc((size_t)(rows > 0 ? rows : 1), sizeof(int64_t));
  int64_t* agree_rows = (int64_t*)calloc((size_t)((rows > 0 ? rows : 1) * (P > 0 ? P : 1)), sizeof(int64_t));
  if (!loss_rows || !correct_rows || !agree_rows) { free(loss_rows); free(correct_rows); free(agree_rows); return 1; }

#ifdef _OPENMP
  if (nthreads <= 0) nthreads = omp_get_max_threads();
#pragma omp parallel num_threads(nthreads)
#endif
  {
    double* z = (double*)malloc(sizeof(double) * (size_t)C);     /* own logits of the row            */
    double* zj = (double*)malloc(sizeof(double) * (size_t)C);    /* one peer's logits                 */
    double* zbar = (double*)malloc(sizeof(double) * (size_t)C);  /* mean of the peers' logits         */
    double* dD = (double*)malloc(sizeof(double) * (size_t)C);    /* dD/dz_c                           */
    double* tmp = (double*)malloc(sizeof(double) * (size_t)C);   /* scaled logits for the KL form     */
#ifdef _OPENMP
#pragma omp for schedule(dynamic, 4)
#endif
    for (int64_t r = 0; r < rows; ++r) {
      int bad = 0;
      const int valid = row_is_valid(labels, mask, r, C, &bad);
      const int want_grad = (grad != NULL && r >= grad_begin && r < grad_end);
      double* g = want_grad ? grad + (size_t)(r - grad_begin) * (size_t)C : NULL;
      if (!valid) { /* masked row: no loss, zero gradient, no counts */
        if (g) for (int64_t c = 0; c < C; ++c) g[c] = 0.0;
        continue;
      }
      const int64_t y = labels[r];
      for (int64_t c = 0; c < C; ++c) z[c] = load_elem(own, dtype, r * row_stride + c);

      /* task loss: cross-entropy against q = (1-eps) onehot(y) + eps/C */
      int64_t a_own = 0;
      const double lse = log_sum_exp(z, C, &a_own);
      double ce = 0.0;
      for (int64_t c = 0; c < C; ++c) {
        const double q = (1.0 - eps) * (c == y ? 1.0 : 0.0) + eps / (double)C;
        ce -= q * (z[c] - lse); /* - sum_c q_c log p_c */
      }
      correct_rows[r] = (a_own == y);

      /* distillation distance and its derivative with respect to z */
      double D = 0.0;
      for (int64_t c = 0; c < C; ++c) { dD[c] = 0.0; zbar[c] = 0.0; }
      if (P >= 1) {
        double lse_own_T = 0.0;
        const int kl_family_kind = dist_kind == ORACLE_DIST_KL || dist_kind == ORACLE_DIST_KL_REVERSE || dist_kind == ORACLE_DIST_KL_SYMMETRIC;
        const double wf = dist_kind == ORACLE_DIST_KL ? 1.0 : dist_kind == ORACLE_DIST_KL_SYMMETRIC ? 0.5 : 0.0;
        const double wr = dist_kind == ORACLE_DIST_KL_REVERSE ? 1.0 : dist_kind == ORACLE_DIST_KL_SYMMETRIC ? 0.5 : 0.0;
        if (kl_family_kind) {
          for (int64_t c = 0; c < C; ++c) tmp[c] = z[c] / T;
          lse_own_T = log_sum_exp(tmp, C, NULL);
        }
        for (int j = 0; j < P; ++j) {
          for (int64_t c = 0; c < C; ++c) zj[c] = load_elem(peers[j], dtype, r * row_stride + c);
          int64_t a_j = 0;
          double mj = zj[0];
          for (int64_t c = 1; c < C; ++c) if (zj[c] > mj) { mj = zj[c]; a_j = c; }
          agree_rows[r * P + j] = (a_j == a_own);
          if (!with_term) continue;
          for (int64_t c = 0; c < C; ++c) zbar[c] += zj[c] / (double)P;
          if (peer_reduce == ORACLE_PEERS_PAIRWISE) {
            if (dist_kind == ORACLE_DIST_MSE_CENTRED) {
              /* both logit vectors centred on their class means: D_j = 1/C sum_c ((z_c - mean z) - (z^(j)_c - mean z^(j)))^2 */
              double mz = 0.0, mj_mean = 0.0;
              for (int64_t c = 0; c < C; ++c) { mz += z[c]; mj_mean += zj[c]; }
              mz /= (double)C; mj_mean /= (double)C;
              double dj = 0.0;
              for (int64_t c = 0; c < C; ++c) {
                const double d = (z[c] - mz) - (zj[c] - mj_mean);
                dj += d * d;
                /* d(D_j)/dz_c = 2/C (d_c - mean_c d) and mean_c d = 0 after centring */
                dD[c] += (2.0 / (double)C) * d / (double)P;
              }
              D += dj / (double)C / (double)P;
            } else if (dist_kind == ORACLE_DIST_MSE) {
              /* D_j = 1/C sum_c (z_c - z^(j)_c)^2 */
              double dj = 0.0;
              for (int64_t c = 0; c < C; ++c) {
                const double d = z[c] - zj[c];
                dj += d * d;
                dD[c] += (2.0 / (double)C) * d / (double)P;
              }
              D += dj / (double)C / (double)P;
            } else {
              /* D_j = T^2 KL(t^(j) || p^T), t^(j) = softmax(z^(j)/T), p^T = softmax(z/T), or its other direction */
              D += kl_family(z, zj, C, T, lse_own_T, wf, wr, 1.0 / (double)P, dD, tmp) / (double)P;
            }
          }
        }
        if (with_term && peer_reduce == ORACLE_PEERS_MEAN_TARGET) {
          if (dist_kind == ORACLE_DIST_MSE_CENTRED) {
            double mz = 0.0, mb = 0.0;
            for (int64_t c = 0; c < C; ++c) { mz += z[c]; mb += zbar[c]; }
            mz /= (double)C; mb /= (double)C;
            double d2 = 0.0;
            for (int64_t c = 0; c < C; ++c) {
              const double d = (z[c] - mz) - (zbar[c] - mb);
              d2 += d * d;
              dD[c] = (2.0 / (double)C) * d;
            }
            D = d2 / (double)C;
          } else if (dist_kind == ORACLE_DIST_MSE) {
            double d2 = 0.0;
            for (int64_t c = 0; c < C; ++c) {
              const double d = z[c] - zbar[c];
              d2 += d * d;
              dD[c] = (2.0 / (double)C) * d;
            }
            D = d2 / (double)C;
          } else {
            D = kl_family(z, zbar, C, T, lse_own_T, wf, wr, 1.0, dD, tmp);
          }
        }
      }

      loss_rows[r] = with_term ? ce + alpha * D : ce;
      if (g) {
        for (int64_t c = 0; c < C; ++c) {
          const double p = exp(z[c] - lse);
          const double q = (1.0 - eps) * (c == y ? 1.0 : 0.0) + eps / (double)C;
          g[c] = w * ((p - q) + (with_term ? alpha * dD[c] : 0.0));
        }
      }
    }
    free(z); free(zj); free(zbar); free(dD); free(tmp);
  }

  /* reduction over rows in index order */
  double total = 0.0;
  int64_t n_correct = 0;
  for (int64_t r = 0; r < rows; ++r) { total += loss_rows[r]; n_correct += correct_rows[r]; }
  if (reduced_loss) *reduced_loss = total * w;
  if (row_loss) for (int64_t r = 0; r < rows; ++r) row_loss[r] = loss_rows[r];
  if (counters) {
    counters[0] = n_valid;
    counters[1] = n_masked;
    counters[2] = n_correct;
    for (int j = 0; j < P; ++j) {
      int64_t s = 0;
      for (int64_t r = 0; r < rows; ++r) s += agree_rows[r * P + j];
      counters[3 + j] = s;
    }
  }
  if (status) *status = any_bad ? ORACLE_STATUS_BAD_LABEL : 0;
  free(loss_rows); free(correct_rows); free(agree_rows);
  return 0;
}
