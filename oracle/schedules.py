"""TEST INFRASTRUCTURE -- plain restatement of the host-side schedules that sit either side of the
loss call in the paper's training recipes, and of Section 3's communication cost model.

Only ``tests/`` may import this module.  Pure Python, written from the definitions:

* penalty coefficient: alpha^k grows by a factor gamma per epoch (appendix, "Neural Machine Translation
  Experiments": gamma = 1.1; "ImageNet Experiments": constant, gamma = 1);
* piecewise-constant schedules over epochs: the learning rate multiplied by 0.1 at each of three
  milestones (Section 4.1; milestones 18, 38, 44 in the tuned schedule, 15, 30, 40 in the original
  one, appendix), the L2 coefficient set to 5e-4, then 1e-5 after the first learning-rate decay and 0
  after the second (Section 4.1), label smoothing decayed / removed the same way (Section 4.2);
* exchange steps: predictions (or checkpoints) are communicated every T iterations, the distillation
  term is left out otherwise (Section 3);
* bits per device and iteration (Section 3): all_reduce 2 b_model, checkpoints (n-1) b_model / T,
  predictions (n-1) b_pred B / T, with b_pred = classes x bits per value.
"""
from __future__ import annotations


def alpha_at_epoch(alpha0: float, gamma: float, epoch: int) -> float:
    a = float(alpha0)
    for _ in range(max(int(epoch), 0)):
        a *= float(gamma)
    return a


def piecewise_constant(values, milestones, epoch: int) -> float:
    """values[0] before the first milestone, values[k] from milestone k-1 on (milestones ascending)."""
    assert len(values) == len(milestones) + 1
    k = 0
    for m in milestones:
        if epoch >= m:
            k += 1
    return float(values[k])


def step_decay(base: float, factor: float, milestones, epoch: int) -> float:
    v = float(base)
    for m in milestones:
        if epoch >= m:
            v *= float(factor)
    return v


def is_exchange_step(step: int, period: int) -> bool:
    return period >= 1 and step % period == 0


def bits_all_reduce(b_model: float) -> float:
    return 2.0 * b_model


def bits_checkpoints(n: int, b_model: float, period: int) -> float:
    return (n - 1) * b_model / period


def bits_predictions(n: int, classes: int, bits_per_value: int, batch_per_device: int, period: int) -> float:
    return (n - 1) * (classes * bits_per_value) * batch_per_device / period
