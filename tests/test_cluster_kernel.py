"""GPU parity of the cluster-resident kernel (all n row images of a row index kept in the shared memory
of a thread-block cluster): every cluster size, both call forms (single model / all models), every
distance it serves, rows that straddle the CTAs' column ranges in all the awkward ways (unaligned rows,
ragged first and last segments, ranges that end up empty), planted maxima on range boundaries.  The kernel
is asked for through CODISTILL_REGIME=cluster; by default it serves only the peer counts the other long-row
kernels are not built for."""
import numpy as np
import pytest
import torch

from paper_2010_02838_b200 import binding as cb
from paper_2010_02838_b200 import synth

from helpers import compare
from test_all_models import compare_all

pytestmark = pytest.mark.gpu


def rand_models(seed, rows, C, n, dtype, scale=1.5, spread=0.7):
    g = np.random.default_rng(seed)
    base = (scale * g.standard_normal((rows, C))).astype(np.float32)
    models = [base + (spread * g.standard_normal((rows, C))).astype(np.float32) for _ in range(n)]
    labels = g.integers(0, C, rows).astype(np.int32)
    labels[0], labels[1], labels[2] = 0, C - 1, C // 2
    if dtype == "bf16":
        models = [synth.f32_to_bf16_bits(m) for m in models]
    mask = (g.random(rows) > 0.1).astype(np.uint8)
    mask[3:5] = 0
    mask[0:3] = 1
    return models, labels, mask


@pytest.fixture(params=[1, 2, 4, 8, 16])
def cluster_size(request, monkeypatch):
    monkeypatch.setenv("CODISTILL_REGIME", "cluster")
    monkeypatch.setenv("CODISTILL_CLUSTER_SIZE", str(request.param))
    return request.param


@pytest.mark.parametrize("n,C,dtype", [(2, 8192, "bf16"), (3, 9001, "bf16"), (8, 5003, "bf16"), (4, 4099, "f32"),
                                       (5, 4100, "bf16"), (2, 2050, "f32")])
def test_single_model_call_every_cluster_size(cluster_size, n, C, dtype):
    rows = 150
    models, labels, mask = rand_models(31 * n + C + cluster_size, rows, C, n, dtype)
    own, peers = models[0], models[1:]
    for dist, pr, T, red in ((cb.DIST_KL_SOFTMAX, cb.PEERS_PAIRWISE_MEAN, 1.0, cb.REDUCE_SUM),
                             (cb.DIST_KL_SOFTMAX, cb.PEERS_PAIRWISE_MEAN, 2.0, cb.REDUCE_MEAN_VALID),
                             (cb.DIST_KL_SOFTMAX, cb.PEERS_MEAN_TARGET, 1.0, cb.REDUCE_SUM),
                             (cb.DIST_KL_SOFTMAX, cb.PEERS_MEAN_TARGET, 0.7, cb.REDUCE_SUM),
                             (cb.DIST_MSE_CENTRED, cb.PEERS_PAIRWISE_MEAN, 1.0, cb.REDUCE_SUM),
                             (cb.DIST_MSE_CENTRED, cb.PEERS_MEAN_TARGET, 1.0, cb.REDUCE_MEAN_VALID)):
        compare(own, peers, labels, mask, alpha=0.9, temperature=T, label_smoothing=0.05, dist=dist, peer_reduce=pr,
                reduction=red, expect_regime="cluster")


@pytest.mark.parametrize("n,C,dtype", [(2, 8192, "bf16"), (8, 5003, "bf16"), (3, 4099, "f32")])
def test_plain_mse_on_request(cluster_size, n, C, dtype):
    rows = 150
    models, labels, mask = rand_models(37 * n + C, rows, C, n, dtype)
    for pr in (cb.PEERS_PAIRWISE_MEAN, cb.PEERS_MEAN_TARGET):
        compare(models[0], models[1:], labels, mask, alpha=0.9, label_smoothing=0.05, peer_reduce=pr,
                reduction=cb.REDUCE_SUM, expect_regime="cluster")


@pytest.mark.parametrize("n,C,dtype", [(2, 8192, "bf16"), (4, 9001, "bf16"), (8, 5003, "bf16"), (3, 4099, "f32")])
def test_all_models_call_every_cluster_size(cluster_size, n, C, dtype):
    rows = 150
    models, labels, mask = rand_models(41 * n + C + cluster_size, rows, C, n, dtype)
    for dist, pr, T, red in ((cb.DIST_MSE_LOGITS, cb.PEERS_PAIRWISE_MEAN, 1.0, cb.REDUCE_SUM),
                             (cb.DIST_MSE_LOGITS, cb.PEERS_MEAN_TARGET, 1.0, cb.REDUCE_MEAN_VALID),
                             (cb.DIST_MSE_CENTRED, cb.PEERS_PAIRWISE_MEAN, 1.0, cb.REDUCE_SUM),
                             (cb.DIST_KL_SOFTMAX, cb.PEERS_PAIRWISE_MEAN, 1.0, cb.REDUCE_SUM),
                             (cb.DIST_KL_SOFTMAX, cb.PEERS_PAIRWISE_MEAN, 2.0, cb.REDUCE_MEAN_VALID)):
        compare_all(models, labels, mask, alpha=0.8, label_smoothing=0.1, peer_reduce=pr, reduction=red, dist=dist,
                    temperature=T)


@pytest.mark.parametrize("n", [5, 6, 7])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_four_to_six_peers_stay_on_a_long_row_kernel(n, dtype):
    """The staged and direct-load kernels are built for 0-3 and 7 peers; the peer counts between are served by
    the cluster-resident kernel (by default), not by the one-CTA-per-row fallback."""
    rows, C = 300, 9001 if dtype == "bf16" else 4099
    models, labels, mask = rand_models(43 * n, rows, C, n, dtype)
    for dist, pr in ((cb.DIST_MSE_LOGITS, cb.PEERS_PAIRWISE_MEAN), (cb.DIST_MSE_LOGITS, cb.PEERS_MEAN_TARGET),
                     (cb.DIST_KL_SOFTMAX, cb.PEERS_PAIRWISE_MEAN), (cb.DIST_MSE_CENTRED, cb.PEERS_PAIRWISE_MEAN)):
        compare(models[0], models[1:], labels, mask, alpha=0.9, temperature=1.5, label_smoothing=0.05, dist=dist,
                peer_reduce=pr, reduction=cb.REDUCE_SUM, expect_regime="cluster")


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_maxima_on_range_boundaries(cluster_size, dtype):
    """Equal maxima planted in the last column of one CTA's range and the first column of the next, on the
    first and last column of an unaligned row, and -0.0 against +0.0: the first arg-max decides every
    counter, bit for bit."""
    rows, C, n = 48, 9003 if dtype == "bf16" else 4611, 3
    V = 8 if dtype == "bf16" else 4
    models, labels, _ = rand_models(5, rows, C, n, dtype, scale=1.0, spread=0.3)
    n_seg = (C + V - 1 + V - 1) // V
    spc = (n_seg + cluster_size - 1) // cluster_size

    def plant(a, r, cols, val):
        v = np.float32(val)
        for c in cols:
            if 0 <= c < C:
                a[r, c] = synth.f32_to_bf16_bits(np.array([v], dtype=np.float32))[0] if a.dtype == np.uint16 else v
    for r in range(rows):
        k = 1 + r % max(cluster_size - 1, 1)
        edge = k * spc * V - (r * C) % V           # first column of CTA k's range in row r
        cols = [edge - 1, edge, C - 1 - (r % 2), r % 3]
        plant(models[0], r, cols, 9.0)
        plant(models[1], r, cols[1:], 9.0)          # ties later: agrees only if its first maximum is the own arg-max
        plant(models[2], r, [min(c for c in cols if 0 <= c < C)], 9.0)
    zero_row = rows - 1                              # all maxima are zeros of either sign
    for m in models:
        m[zero_row] = (synth.f32_to_bf16_bits(np.full(C, -1.0, dtype=np.float32)) if m.dtype == np.uint16
                       else np.full(C, -1.0, dtype=np.float32))
    plant(models[0], zero_row, [7, 4000], -0.0)
    plant(models[0], zero_row, [2000], 0.0)
    plant(models[1], zero_row, [7], 0.0)
    plant(models[2], zero_row, [2000], -0.0)
    compare(models[0], models[1:], labels, None, alpha=1.0, dist=cb.DIST_MSE_CENTRED, reduction=cb.REDUCE_SUM,
            expect_regime="cluster")
    compare_all(models, labels, None, alpha=1.0, reduction=cb.REDUCE_SUM)


def test_guard_bands_and_determinism(monkeypatch):
    """Nothing is written outside the gradient rows (an unaligned last row ends inside a 16-byte segment),
    two runs are bit-identical, inputs are left alone."""
    monkeypatch.setenv("CODISTILL_REGIME", "cluster")
    rows, C, n = 40, 9001, 4
    models, labels, mask = rand_models(9, rows, C, n, "bf16")
    keep = [m.copy() for m in models]
    plan, out, _ = compare(models[0], models[1:], labels, mask, alpha=1.0, temperature=2.0, dist=cb.DIST_KL_SOFTMAX,
                           reduction=cb.REDUCE_SUM, expect_regime="cluster")
    g = torch.full((rows * C + 64,), 3.0, dtype=torch.bfloat16, device="cuda")
    plan.params.grad_logits = g[32:].data_ptr()
    first = (out.grad.clone(), out.row_loss.clone(), out.loss.clone(), out.counters.clone())
    plan.run()
    torch.cuda.synchronize()
    assert torch.all(g[:32].float() == 3.0) and torch.all(g[32 + rows * C:].float() == 3.0)
    assert torch.equal(g[32:32 + rows * C].view(rows, C), first[0])
    assert torch.equal(first[1], out.row_loss) and torch.equal(first[2], out.loss) and torch.equal(first[3], out.counters)
    for m, k in zip(models, keep):
        assert np.array_equal(m, k)
