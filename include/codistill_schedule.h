/*
 * codistill_schedule.h -- host-side schedules that sit either side of the loss call in the
 * training recipes of "A Closer Look at Codistillation for Distributed Training" (arXiv
 * 2010.02838), and Section 3's communication cost model.  Plain host arithmetic: no device
 * work, no state, no allocation; every function is reentrant.
 */
#ifndef CODISTILL_SCHEDULE_H_
#define CODISTILL_SCHEDULE_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/*
 * Penalty coefficient alpha^k of Algorithm 1 at a given epoch: alpha0 * gamma^epoch.  The appendix
 * ("Neural Machine Translation Experiments") grows alpha by gamma = 1.1 every epoch; the ImageNet
 * experiments keep it constant (gamma = 1, alpha0 = 1).  epoch < 0 counts as 0.  NaN when alpha0 or
 * gamma is not finite.
 */
double codistill_schedule_alpha(double alpha0, double gamma, int64_t epoch);

/*
 * Piecewise-constant schedule over epochs: values[0] before milestones[0], values[k] from
 * milestones[k-1] on.  `values` has n_milestones + 1 entries; milestones must be ascending.  This is
 * the form of Section 4.1's L2 schedule (5e-4, then 1e-5 after the first learning-rate decay, 0 after
 * the second: values {5e-4, 1e-5, 0}, milestones = the first two learning-rate milestones) and of
 * Section 4.2's decayed / removed label smoothing.  HOST pointers, read only.  NaN on NULL pointers,
 * n_milestones < 0 or milestones out of order.
 */
double codistill_schedule_piecewise(const double* values, const int64_t* milestones, int n_milestones, int64_t epoch);

/*
 * Step-wise decay: base * factor^(number of milestones <= epoch).  Section 4.1 decreases the learning
 * rate three times by 0.1; the appendix moves the milestones from {15, 30, 40} to {18, 38, 44} for
 * codistillation.  NaN on NULL milestones with n_milestones > 0 or n_milestones < 0.
 */
double codistill_schedule_step_decay(double base, double factor, const int64_t* milestones, int n_milestones, int64_t epoch);

/*
 * Section 3: predictions (or checkpoints) are communicated every `period` iterations and the
 * distillation term is left out on the others.  Returns 1 when iteration `step` (0-based) is a
 * communication step, else 0 (also for period < 1 or step < 0): on a 0 the caller runs the loss with
 * n = 1 (or alpha = 0), which skips the peers entirely.
 */
int codistill_is_exchange_step(int64_t step, int64_t period);

/*
 * Section 3's cost model, bits sent per device and iteration (averaged over a period):
 *   all_reduce                        2 * b_model
 *   checkpoints every `period`        (n - 1) * b_model / period
 *   predictions every `period`        (n - 1) * b_pred * batch_per_device / period,
 *                                     b_pred = classes * bits_per_value  (3.2e4 for 1000 classes, 32 bit)
 * NaN on n < 1, period < 1 or negative sizes.
 */
double codistill_bits_all_reduce(double b_model);
double codistill_bits_checkpoints(int n, double b_model, int64_t period);
double codistill_bits_predictions(int n, int64_t classes, int bits_per_value, int64_t batch_per_device, int64_t period);

#ifdef __cplusplus
}
#endif
#endif /* CODISTILL_SCHEDULE_H_ */
