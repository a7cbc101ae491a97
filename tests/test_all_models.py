"""GPU parity of the all-models call (Algorithm 1's loop over the n models on one minibatch): every
model's loss, gradient and counters against the oracle's single-model definition evaluated n times."""
import numpy as np
import pytest
import torch

import oracle
from paper_2010_02838_b200 import binding as cb
from paper_2010_02838_b200 import synth

from helpers import TOL, bf16_round, bf16_ulp, grad_to_f64, to_device

pytestmark = pytest.mark.gpu


def rand_models(seed, rows, C, n, dtype, scale=1.5, spread=0.7):
    g = np.random.default_rng(seed)
    base = scale * g.standard_normal((rows, C))
    models = [(base + spread * g.standard_normal((rows, C))).astype(np.float32) for _ in range(n)]
    labels = g.integers(0, C, rows).astype(np.int32)
    if dtype == "bf16":
        models = [synth.f32_to_bf16_bits(m) for m in models]
    return models, labels


def compare_all(models, labels, mask, *, classes=None, alpha=1.0, label_smoothing=0.0, peer_reduce=0, reduction=0, dist=0,
                temperature=1.0):
    kind = "f32" if models[0].dtype == np.float32 else "bf16"
    tol = TOL[kind]
    C = models[0].shape[1] if classes is None else classes
    d_models = [to_device(m) for m in models]
    views = [m[:, :C] for m in d_models] if C != models[0].shape[1] else d_models
    plan = cb.AllPlan(views, to_device(labels), to_device(mask), classes=classes, alpha=alpha,
                      label_smoothing=label_smoothing, peer_reduce=peer_reduce, reduction=reduction, dist=dist,
                      temperature=temperature)
    out = plan.run()
    torch.cuda.synchronize()
    refs = oracle.codistill_all(models, labels, mask, classes=classes, alpha=alpha, label_smoothing=label_smoothing,
                                peer_reduce=peer_reduce, reduction=reduction, dist=dist, temperature=temperature)
    counters = out.counters.cpu().numpy()
    losses = out.loss.cpu().numpy()
    rows_loss = out.row_loss.cpu().numpy().astype(np.float64)
    for i, ref in enumerate(refs):
        assert int(out.status.item()) == ref.status
        assert counters[i].tolist() == ref.counters.tolist(), (i, counters[i], ref.counters)   # integers: bit-exact
        assert abs(losses[i] - ref.loss) <= tol["loss_rel"] * abs(ref.loss) + tol["loss_floor"], (i, losses[i], ref.loss)
        np.testing.assert_allclose(rows_loss[i], ref.row_loss, rtol=tol["loss_rel"], atol=tol["loss_floor"])
        g = grad_to_f64(out.grads[i])[:, :C]
        err = np.abs(g - ref.grad)
        if kind == "f32":
            assert err.max(initial=0.0) <= tol["grad_abs"], (i, err.max())
        else:
            bound = np.maximum(tol["grad_abs"], 0.75 * bf16_ulp(ref.grad))
            assert np.all(err <= bound), (i, float((err - bound).max()))
            scale = 1.0 if reduction == cb.REDUCE_SUM else 1.0 / max(int(ref.counters[0]), 1)
            step = bf16_ulp(np.maximum(np.abs(ref.grad), np.abs(g)))
            assert np.all(np.abs(g - bf16_round(ref.grad)) <= step * 1.0001 + 1e-6 * scale)
    return plan, out, refs


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("n", [2, 3, 4, 5, 8])
@pytest.mark.parametrize("C", [10, 1000, 4099, 9001])
def test_all_models_parity(dtype, n, C):
    rows = 19
    models, labels = rand_models(100 * n + C, rows, C, n, dtype)
    mask = (np.arange(rows) % 7 != 3).astype(np.uint8)
    labels[0], labels[1] = 0, C - 1
    for peer_reduce, reduction, dist in ((cb.PEERS_PAIRWISE_MEAN, cb.REDUCE_SUM, cb.DIST_MSE_LOGITS),
                                         (cb.PEERS_MEAN_TARGET, cb.REDUCE_MEAN_VALID, cb.DIST_MSE_LOGITS),
                                         (cb.PEERS_PAIRWISE_MEAN, cb.REDUCE_SUM, cb.DIST_MSE_CENTRED),
                                         (cb.PEERS_MEAN_TARGET, cb.REDUCE_SUM, cb.DIST_MSE_CENTRED)):
        compare_all(models, labels, mask, alpha=0.8, label_smoothing=0.1, peer_reduce=peer_reduce, reduction=reduction,
                    dist=dist)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("n", [2, 3, 5, 8])
@pytest.mark.parametrize("C", [10, 1000, 4099, 9001])
def test_all_models_kl_parity(dtype, n, C):
    """KL distance, pairwise over the peers, at T = 1 and T != 1."""
    rows = 19
    models, labels = rand_models(300 * n + C, rows, C, n, dtype)
    mask = (np.arange(rows) % 7 != 3).astype(np.uint8)
    labels[0], labels[1] = 0, C - 1
    for temperature, reduction in ((1.0, cb.REDUCE_SUM), (2.0, cb.REDUCE_MEAN_VALID), (0.7, cb.REDUCE_SUM)):
        compare_all(models, labels, mask, alpha=0.8, label_smoothing=0.1, reduction=reduction, dist=cb.DIST_KL_SOFTMAX,
                    temperature=temperature)
    if n == 2:   # two models: the mean target is the one peer
        compare_all(models, labels, mask, alpha=0.8, peer_reduce=cb.PEERS_MEAN_TARGET, reduction=cb.REDUCE_SUM,
                    dist=cb.DIST_KL_SOFTMAX, temperature=2.0)


def test_all_models_kl_limits():
    """Mean target with more than two models is refused; identical models give zero distance; the call
    equals the n single-model KL calls on a workload-shaped row."""
    rows, C, n = 8, 32768, 2
    models, labels = rand_models(77, rows, C, n, "bf16")
    compare_all(models, labels, None, alpha=1.0, reduction=cb.REDUCE_SUM, dist=cb.DIST_KL_SOFTMAX, temperature=2.0)
    models3, labels3 = rand_models(78, 6, 50257, 3, "bf16")
    compare_all(models3, labels3, None, alpha=1.0, reduction=cb.REDUCE_SUM, dist=cb.DIST_KL_SOFTMAX)
    d = [to_device(m) for m in models3]
    with pytest.raises(cb.CodistillError):
        cb.AllPlan(d, to_device(labels3), None, dist=cb.DIST_KL_SOFTMAX, peer_reduce=cb.PEERS_MEAN_TARGET).run()
    with pytest.raises(cb.CodistillError):
        cb.AllPlan(d, to_device(labels3), None, dist=cb.DIST_KL_SOFTMAX, temperature=0.0).run()
    same = [models3[0].copy() for _ in range(3)]
    plan, out, refs = compare_all(same, labels3, None, alpha=2.0, reduction=cb.REDUCE_SUM, dist=cb.DIST_KL_SOFTMAX,
                                  temperature=1.5)
    ce_only = oracle.codistill(same[0], [], labels3, None, reduction=oracle.REDUCE_SUM)
    assert abs(out.loss[0].item() - ce_only.loss) <= 1e-5 * abs(ce_only.loss)
    dl = to_device(labels3)
    allp = cb.AllPlan(d, dl, None, alpha=1.0, temperature=2.0, dist=cb.DIST_KL_SOFTMAX, reduction=cb.REDUCE_SUM).run()
    for i in range(3):
        single = cb.Plan(d[i], d[:i] + d[i + 1:], dl, None, alpha=1.0, temperature=2.0, dist=cb.DIST_KL_SOFTMAX,
                         reduction=cb.REDUCE_SUM).run()
        torch.cuda.synchronize()
        assert single.counters.cpu().tolist() == allp.counters[i].cpu().tolist()
        assert abs(single.loss.item() - allp.loss[i].item()) <= 1e-4 * abs(single.loss.item())


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_all_models_on_workload_shapes(dtype):
    """Unaligned 50257-class rows (n = 8) and 32768-class rows (n = 2) at a few rows; row pitch."""
    for n, C, stride in ((8, 50257, 50257), (2, 32768, 32768), (3, 1000, 1024)):
        rows = 6
        models, labels = rand_models(C + n, rows, stride, n, dtype)
        labels = labels % C
        mask = np.array([1, 1, 0, 1, 1, 1], dtype=np.uint8)
        compare_all(models, labels, mask, classes=C if stride != C else None, alpha=1.0, reduction=cb.REDUCE_SUM)


def test_all_models_ties_and_degenerate_cases():
    """Planted equal maxima (agreement counters), identical models (distance exactly 0), alpha = 0,
    all rows masked, zero rows."""
    rows, C, n = 12, 777, 4
    models, labels = rand_models(9, rows, C, n, "f32", scale=1.0)
    for r in range(rows):
        cols = [(r * 53) % C, (r * 53 + 5) % C]
        for i, m in enumerate(models):
            m[r, cols[0 if i % 2 == 0 else 1]] = 9.0
            if i == 3:
                m[r, cols[0]] = 9.0                      # model 3 ties on both columns: its first arg-max decides
    compare_all(models, labels, None, alpha=1.0, reduction=cb.REDUCE_SUM)
    same = [models[0].copy() for _ in range(3)]
    plan, out, refs = compare_all(same, labels, None, alpha=2.0, reduction=cb.REDUCE_SUM)
    ce_only = oracle.codistill(same[0], [], labels, None, reduction=oracle.REDUCE_SUM)
    assert abs(out.loss[0].item() - ce_only.loss) <= 1e-5 * abs(ce_only.loss)
    compare_all(models, labels, None, alpha=0.0)
    compare_all(models, labels, np.zeros(rows, dtype=np.uint8), alpha=1.0)
    empty = [m[:0] for m in models]
    compare_all(empty, labels[:0], None, alpha=1.0)


def test_all_models_equals_single_calls():
    """Integer outputs identical, losses and gradients within rounding of the n single-model calls."""
    rows, C, n = 40, 8192, 4
    models, labels = rand_models(21, rows, C, n, "bf16")
    mask = (np.arange(rows) % 9 != 0).astype(np.uint8)
    d = [to_device(m) for m in models]
    dl, dm = to_device(labels), to_device(mask)
    allp = cb.AllPlan(d, dl, dm, alpha=1.0, reduction=cb.REDUCE_SUM)
    out = allp.run()
    torch.cuda.synchronize()
    for i in range(n):
        single = cb.Plan(d[i], d[:i] + d[i + 1:], dl, dm, alpha=1.0, reduction=cb.REDUCE_SUM).run()
        torch.cuda.synchronize()
        assert single.counters.cpu().tolist() == out.counters[i].cpu().tolist()
        assert abs(single.loss.item() - out.loss[i].item()) <= 1e-5 * abs(single.loss.item())
        diff = (single.grad.float() - out.grads[i].float()).abs()
        step = torch.maximum(single.grad.float().abs(), out.grads[i].float().abs()) * 2.0 ** -7
        assert bool(torch.all(diff <= step + 1e-6))


def test_all_models_determinism_and_untouched_padding():
    """Two runs are bit-identical; with a row pitch the padding columns of the gradients are never written."""
    rows, C, stride, n = 23, 5001, 5008, 3
    models, labels = rand_models(4, rows, stride, n, "bf16")
    labels = labels % C
    mask = (np.arange(rows) % 4 != 1).astype(np.uint8)
    d = [to_device(m) for m in models]
    plan = cb.AllPlan([m[:, :C] for m in d], to_device(labels), to_device(mask), classes=C, alpha=1.0,
                      reduction=cb.REDUCE_SUM)
    for g in plan.out.grads:   # fill the whole storage, padding columns included
        g.as_strided(((rows - 1) * stride + C,), (1,)).fill_(7.0)
    out = plan.run()
    torch.cuda.synchronize()
    first = ([g.clone() for g in out.grads], out.row_loss.clone(), out.loss.clone(), out.counters.clone())
    out = plan.run()
    torch.cuda.synchronize()
    for g0, g1 in zip(first[0], out.grads):
        assert torch.equal(g0, g1)
        assert g1.stride(0) == stride
        pad = g1.as_strided((rows - 1, stride), (stride, 1))[:, C:]     # the last row has no padding behind it
        assert torch.all(pad.float() == 7.0)
    assert torch.equal(first[1], out.row_loss) and torch.equal(first[2], out.loss) and torch.equal(first[3], out.counters)
