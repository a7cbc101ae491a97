// Host-side schedules and Section 3's communication cost model (include/codistill_schedule.h).
// No device code: this file only rides along in the library.
#include <math.h>

#include "../../include/codistill_schedule.h"

extern "C" {

double codistill_schedule_alpha(double alpha0, double gamma, int64_t epoch) {
  if (!isfinite(alpha0) || !isfinite(gamma)) return NAN;
  double a = alpha0;
  for (int64_t k = 0; k < epoch; ++k) a *= gamma;   // repeated product: the value a trainer that multiplies once per epoch holds
  return a;
}

static int milestones_passed(const int64_t* milestones, int n, int64_t epoch, bool* ordered) {
  int passed = 0;
  *ordered = true;
  for (int k = 0; k < n; ++k) {
    if (k > 0 && milestones[k] < milestones[k - 1]) *ordered = false;
    if (epoch >= milestones[k]) ++passed;
  }
  return passed;
}

double codistill_schedule_piecewise(const double* values, const int64_t* milestones, int n_milestones, int64_t epoch) {
  if (values == nullptr || n_milestones < 0 || (n_milestones > 0 && milestones == nullptr)) return NAN;
  bool ordered;
  const int k = milestones_passed(milestones, n_milestones, epoch, &ordered);
  return ordered ? values[k] : NAN;
}

double codistill_schedule_step_decay(double base, double factor, const int64_t* milestones, int n_milestones, int64_t epoch) {
  if (n_milestones < 0 || (n_milestones > 0 && milestones == nullptr)) return NAN;
  bool ordered;
  const int k = milestones_passed(milestones, n_milestones, epoch, &ordered);
  double v = base;
  for (int i = 0; i < k; ++i) v *= factor;
  return v;
}

int codistill_is_exchange_step(int64_t step, int64_t period) {
  return (period >= 1 && step >= 0 && step % period == 0) ? 1 : 0;
}

double codistill_bits_all_reduce(double b_model) { return b_model >= 0.0 ? 2.0 * b_model : NAN; }

double codistill_bits_checkpoints(int n, double b_model, int64_t period) {
  if (n < 1 || period < 1 || !(b_model >= 0.0)) return NAN;
  return (double)(n - 1) * b_model / (double)period;
}

double codistill_bits_predictions(int n, int64_t classes, int bits_per_value, int64_t batch_per_device, int64_t period) {
  if (n < 1 || period < 1 || classes < 0 || bits_per_value < 0 || batch_per_device < 0) return NAN;
  return (double)(n - 1) * ((double)classes * (double)bits_per_value) * (double)batch_per_device / (double)period;
}

}  // extern "C"
