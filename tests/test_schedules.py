"""Host-side schedules and Section 3's cost model: the plain restatement under oracle/ against the
values the paper prints (tests/golden/schedules_paper_values.txt), then the library's C functions
against that restatement.  No GPU needed: these are host functions."""
import math
import os

import pytest

from oracle import schedules as ref
from paper_2010_02838_b200 import binding as cb
from paper_2010_02838_b200 import build as cbuild

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "schedules_paper_values.txt")


@pytest.fixture(scope="module")
def paper():
    vals = {}
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, *rest = line.split()
        nums = [float(x) for x in rest]
        vals[key] = nums[0] if len(nums) == 1 else nums
    return vals


@pytest.fixture(scope="module", autouse=True)
def built():
    cbuild.build()
    cb.load_library()


# ---------------------------------------------------------------- the restatement against the paper
def test_oracle_l2_schedule_is_the_papers(paper):
    """Section 4.1: 5e-4, then 1e-5 after the first learning-rate decay, 0 after the second."""
    values = [paper["wd_initial"], paper["wd_after_first_decay"], paper["wd_after_second_decay"]]
    ms = [int(m) for m in paper["lr_milestones_tuned"][:2]]
    assert values == [5e-4, 1e-5, 0.0] and ms == [18, 38]
    got = [ref.piecewise_constant(values, ms, e) for e in (0, 17, 18, 37, 38, 44, 89)]
    assert got == [5e-4, 5e-4, 1e-5, 1e-5, 0.0, 0.0, 0.0]


def test_oracle_learning_rate_steps_are_the_papers(paper):
    """Three decreases by 0.1 (Section 4.1) at epochs 18, 38, 44 (appendix; 15, 30, 40 before tuning)."""
    for key, ms in (("lr_milestones_tuned", [18, 38, 44]), ("lr_milestones_original", [15, 30, 40])):
        assert [int(m) for m in paper[key]] == ms
        lr = [ref.step_decay(0.2, paper["lr_factor"], ms, e) for e in (0, ms[0] - 1, ms[0], ms[1], ms[2], 89)]
        assert lr[0] == lr[1] == 0.2
        assert lr[2] == pytest.approx(0.02) and lr[3] == pytest.approx(0.002)
        assert lr[4] == lr[5] == pytest.approx(0.0002)


def test_oracle_alpha_growth_is_the_papers(paper):
    """alpha grows by gamma = 1.1 per epoch on translation, stays 1 on ImageNet."""
    g = paper["alpha_gamma_nmt"]
    assert g == 1.1
    for k in (0, 1, 2, 10, 40):
        assert ref.alpha_at_epoch(1.0, g, k) == pytest.approx(1.1 ** k, rel=1e-12)
    assert ref.alpha_at_epoch(1.0, g, 10) == pytest.approx(2.5937424601, rel=1e-10)   # (11/10)^10 written out
    assert all(ref.alpha_at_epoch(paper["alpha_imagenet"], 1.0, k) == 1.0 for k in range(90))


def test_oracle_cost_model_is_section_3(paper):
    b_model, b_pred, B = paper["b_model"], paper["b_pred"], int(paper["batch_per_gpu"])
    assert ref.bits_all_reduce(b_model) == paper["all_reduce_bits"] == 1.6e9
    assert ref.bits_predictions(2, 1000, 32, 1, 1) == b_pred == 3.2e4          # one sample: 1000 classes x 32 bit
    assert ref.bits_predictions(2, 1000, 32, B, 1) == 1.024e6                  # n = 2, batch 32 per GPU, every step
    assert ref.bits_predictions(2, 1000, 32, B, 100) == 1.024e4
    assert ref.bits_predictions(4, 1000, 32, B, 1) == 3 * 1.024e6
    T = int(paper["checkpoint_period_example"])
    assert ref.bits_checkpoints(2, b_model, T) == 1.6e7
    # Section 3: checkpoints beat all_reduce exactly when (n - 1) / T < 2
    for n, period in ((2, 1), (3, 1), (3, 2), (4, 1), (9, 4), (9, 5)):
        assert (ref.bits_checkpoints(n, b_model, period) < ref.bits_all_reduce(b_model)) == ((n - 1) / period < 2)
    # the headline ratio: predictions every step against all_reduce, ResNet50 / ImageNet
    assert ref.bits_all_reduce(b_model) / ref.bits_predictions(2, 1000, 32, B, 1) == pytest.approx(1562.5)


def test_oracle_exchange_steps():
    assert [s for s in range(12) if ref.is_exchange_step(s, 5)] == [0, 5, 10]
    assert all(ref.is_exchange_step(s, 1) for s in range(5))
    assert not ref.is_exchange_step(3, 0)


# ---------------------------------------------------------------- the library against the restatement
def test_library_alpha_matches():
    for a0, g in ((1.0, 1.1), (0.5, 1.1), (1.0, 1.0), (2.0, 0.9)):
        for k in (-3, 0, 1, 7, 40, 89):
            assert cb.schedule_alpha(a0, g, k) == ref.alpha_at_epoch(a0, g, k)
    assert math.isnan(cb.schedule_alpha(float("inf"), 1.1, 3))


def test_library_piecewise_and_step_decay_match():
    values, ms = [5e-4, 1e-5, 0.0], [18, 38]
    for e in range(-1, 60):
        assert cb.schedule_piecewise(values, ms, e) == ref.piecewise_constant(values, ms, e)
        assert cb.schedule_step_decay(0.2, 0.1, [18, 38, 44], e) == ref.step_decay(0.2, 0.1, [18, 38, 44], e)
    assert cb.schedule_piecewise([0.1], [], 5) == 0.1                       # no milestone: constant
    assert cb.schedule_piecewise([0.1, 0.05, 0.0], [10, 20], 25) == 0.0     # label smoothing removed
    assert math.isnan(cb.schedule_piecewise([1.0, 2.0, 3.0], [20, 10], 5))  # milestones out of order


def test_library_exchange_and_bits_match():
    for period in (1, 5, 10, 100, 0, -2):
        for step in (-1, 0, 1, 4, 5, 99, 100, 1000):
            assert cb.is_exchange_step(step, period) == (step >= 0 and ref.is_exchange_step(step, period))
    assert cb.bits_all_reduce(8e8) == ref.bits_all_reduce(8e8)
    for n, T in ((2, 1), (2, 50), (4, 625), (8, 5000)):
        assert cb.bits_checkpoints(n, 8e8, T) == ref.bits_checkpoints(n, 8e8, T)
        assert cb.bits_predictions(n, 1000, 32, 32, T) == ref.bits_predictions(n, 1000, 32, 32, T)
        assert cb.bits_predictions(n, 32768, 16, 3854, T) == ref.bits_predictions(n, 32768, 16, 3854, T)
    assert math.isnan(cb.bits_checkpoints(0, 8e8, 1)) and math.isnan(cb.bits_predictions(2, 1000, 32, 32, 0))
