"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle, element by element, on
the five seeded synthetic workloads (the two largest here at reduced row counts that still span
several CTAs; their full sizes are covered by test_parity_fullsize.py)."""
import itertools

import numpy as np
import pytest

from paper_2010_02838_b200 import binding as cb
from paper_2010_02838_b200 import synth

from helpers import compare

pytestmark = pytest.mark.gpu

DISTS = [cb.DIST_MSE_LOGITS, cb.DIST_KL_SOFTMAX, cb.DIST_MSE_CENTRED, cb.DIST_KL_REVERSE, cb.DIST_KL_SYMMETRIC]
PEERS = [cb.PEERS_PAIRWISE_MEAN, cb.PEERS_MEAN_TARGET]
REDS = [cb.REDUCE_SUM, cb.REDUCE_MEAN_VALID]


def workload(idx):
    w = synth.WORKLOADS[idx]
    if idx == 4:
        return synth.scaled(w, rows=320)        # 10 sentences x 32 tokens, 32 padded rows
    if idx == 5:
        return synth.scaled(w, rows=160)
    return w


@pytest.mark.parametrize("idx", [1, 2, 3, 4, 5])
@pytest.mark.parametrize("dist,pr,red", list(itertools.product(DISTS, PEERS, REDS)))
def test_workload_parity(idx, dist, pr, red):
    w = workload(idx)
    own, peers, labels, mask = synth.make_inputs(w)
    plan, _, _ = compare(own, peers, labels, mask, alpha=w.alpha, temperature=w.temperature,
                         label_smoothing=w.label_smoothing, dist=dist, peer_reduce=pr, reduction=red)
    if dist == cb.DIST_MSE_LOGITS:   # which kernel served the workload
        assert plan.regime == {1: "short", 2: "short", 3: "short", 4: "tma", 5: "stream"}[idx]


@pytest.mark.parametrize("idx,regime", [(4, "stream"), (5, "tma")])
@pytest.mark.parametrize("pr,red", list(itertools.product(PEERS, REDS)))
def test_workload_parity_other_long_row_kernel(monkeypatch, idx, regime, pr, red):
    """The two largest workloads on the long-row kernel that is not their default."""
    monkeypatch.setenv("CODISTILL_REGIME", regime)
    w = workload(idx)
    own, peers, labels, mask = synth.make_inputs(w)
    compare(own, peers, labels, mask, alpha=w.alpha, temperature=w.temperature, label_smoothing=w.label_smoothing,
            dist=cb.DIST_MSE_LOGITS, peer_reduce=pr, reduction=red, expect_regime=regime)


@pytest.mark.parametrize("idx", [1, 2, 3])
@pytest.mark.parametrize("pr,red", list(itertools.product(PEERS, REDS)))
def test_short_workloads_on_the_two_launch_kernel(monkeypatch, idx, pr, red):
    """The three small workloads on the warp-per-row kernel behind a counting launch (their default is the
    single-launch kernel)."""
    monkeypatch.setenv("CODISTILL_REGIME", "warp")
    w = workload(idx)
    own, peers, labels, mask = synth.make_inputs(w)
    compare(own, peers, labels, mask, alpha=w.alpha, temperature=w.temperature, label_smoothing=w.label_smoothing,
            dist=cb.DIST_MSE_LOGITS, peer_reduce=pr, reduction=red, expect_regime="warp")


@pytest.mark.parametrize("idx", [1, 2, 3])
def test_every_model_role(idx):
    """One call serves one model; relabelling which tensor is 'own' serves all n models."""
    w = workload(idx)
    models = [synth.make_model_logits(w, k) for k in range(w.n)]
    labels = synth.make_labels(w)
    for i in range(w.n):
        compare(models[i], models[:i] + models[i + 1:], labels, None, alpha=w.alpha, reduction=cb.REDUCE_SUM)


def test_basic_entry_point_matches_oracle():
    """codistill_loss_fwd_bwd: MSE distance, mean over valid rows, scratch from the stream-ordered allocator."""
    import torch
    import oracle
    from helpers import to_device
    w = synth.WORKLOADS[2]
    own, peers, labels, _ = synth.make_inputs(w)
    mask = (np.arange(w.rows) % 7 != 0).astype(np.uint8)
    for _ in range(2):
        out = cb.codistill_loss_fwd_bwd(to_device(own), [to_device(p) for p in peers], to_device(labels),
                                        to_device(mask), alpha=0.7, temperature=3.0)
        torch.cuda.synchronize()
        ref = oracle.codistill(own, peers, labels, mask, alpha=0.7)
        assert abs(out.loss.item() - ref.loss) <= 1e-5 * abs(ref.loss)
        np.testing.assert_allclose(out.row_loss.cpu().numpy(), ref.row_loss, rtol=1e-5, atol=1e-7)
        assert np.abs(out.grad.double().cpu().numpy() - ref.grad).max() <= 1e-6
