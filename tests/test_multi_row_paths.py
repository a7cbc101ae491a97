"""GPU parity of the persistent long-row kernels in their multi-row mode.

The long-row kernels run a fixed number of CTAs (a few per SM) that draw rows from a counter, so
with more rows than CTAs every CTA works through several rows in turn: it alternates between two
sets of partial-result buffers, hands the next row id over between rows and meets masked rows
between valid ones.  The batches here hold at least three rows per CTA slot of a 148-SM device (592
slots at most), with a mask that scatters padded rows among valid ones, and are compared with the
oracle element by element: softmax-KL distance, centred MSE distance, the all-models call and the
host-buffer entry point with slices taller than the number of slots.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2010_02838_b200 import binding as cb
from paper_2010_02838_b200 import synth

from helpers import TOL, bf16_ulp, compare, to_device
from test_all_models import compare_all

pytestmark = pytest.mark.gpu

ROWS = 1800          # > 3 x 592 CTA slots


def rand_models(seed, rows, C, n, dtype, scale=1.5, spread=0.7):
    """n models = shared base + per-model noise (float32 or bf16 bits), labels, scattered mask."""
    g = np.random.default_rng(seed)
    base = (scale * g.standard_normal((rows, C))).astype(np.float32)
    models = [base + (spread * g.standard_normal((rows, C))).astype(np.float32) for _ in range(n)]
    labels = g.integers(0, C, rows).astype(np.int32)
    labels[0], labels[1] = 0, C - 1
    if dtype == "bf16":
        models = [synth.f32_to_bf16_bits(m) for m in models]
    # padded rows among valid ones: single rows, pairs, and a run of five (so that a CTA meets
    # masked rows back to back), none of them periodic in the number of CTAs
    mask = (g.random(rows) > 0.12).astype(np.uint8)
    mask[7:12] = 0
    mask[rows - 1] = 0
    mask[0] = 1
    return models, labels, mask


@pytest.mark.parametrize("n,C,dtype,peer_reduce,temperature", [
    (2, 8192, "bf16", cb.PEERS_PAIRWISE_MEAN, 1.0),
    (2, 9001, "bf16", cb.PEERS_MEAN_TARGET, 2.0),
    (4, 9001, "bf16", cb.PEERS_PAIRWISE_MEAN, 0.7),
    (4, 8192, "bf16", cb.PEERS_MEAN_TARGET, 1.0),
    (8, 9001, "bf16", cb.PEERS_PAIRWISE_MEAN, 2.0),
    (8, 8200, "bf16", cb.PEERS_MEAN_TARGET, 1.0),
    (4, 4099, "f32", cb.PEERS_PAIRWISE_MEAN, 1.5),
    (3, 5000, "bf16", cb.PEERS_PAIRWISE_MEAN, 1.0),
    (6, 4501, "bf16", cb.PEERS_PAIRWISE_MEAN, 1.3),
])
def test_kl_many_rows_per_cta(n, C, dtype, peer_reduce, temperature):
    models, labels, mask = rand_models(11 * n + C, ROWS, C, n, dtype)
    for reduction in (cb.REDUCE_SUM, cb.REDUCE_MEAN_VALID):
        compare(models[0], models[1:], labels, mask, alpha=0.9, temperature=temperature, label_smoothing=0.05,
                dist=cb.DIST_KL_SOFTMAX, peer_reduce=peer_reduce, reduction=reduction)


@pytest.mark.parametrize("n,C,dtype,peer_reduce", [
    (2, 8192, "bf16", cb.PEERS_PAIRWISE_MEAN),
    (4, 9001, "bf16", cb.PEERS_MEAN_TARGET),
    (8, 9001, "bf16", cb.PEERS_PAIRWISE_MEAN),
    (3, 4099, "f32", cb.PEERS_PAIRWISE_MEAN),
    (6, 4501, "bf16", cb.PEERS_MEAN_TARGET),
])
def test_centred_mse_many_rows_per_cta(n, C, dtype, peer_reduce):
    models, labels, mask = rand_models(13 * n + C, ROWS, C, n, dtype)
    if dtype == "f32":   # class means that differ between the models
        models = [m + np.float32(0.5 * j) for j, m in enumerate(models)]
    for reduction in (cb.REDUCE_SUM, cb.REDUCE_MEAN_VALID):
        compare(models[0], models[1:], labels, mask, alpha=0.9, label_smoothing=0.05, dist=cb.DIST_MSE_CENTRED,
                peer_reduce=peer_reduce, reduction=reduction)


@pytest.mark.parametrize("n,C,dtype", [(2, 8192, "bf16"), (8, 9001, "bf16"), (5, 4400, "bf16"), (3, 4099, "f32")])
def test_plain_mse_many_rows_per_cta(monkeypatch, n, C, dtype):
    """The direct-load kernel with the plain MSE distance, forced where the staged kernel is the default."""
    monkeypatch.setenv("CODISTILL_REGIME", "stream")
    models, labels, mask = rand_models(17 * n + C, ROWS, C, n, dtype)
    compare(models[0], models[1:], labels, mask, alpha=0.9, label_smoothing=0.05, reduction=cb.REDUCE_SUM)


@pytest.mark.parametrize("n,C,dtype", [(2, 8192, "bf16"), (4, 9001, "bf16"), (8, 9001, "bf16"), (3, 4099, "f32")])
@pytest.mark.parametrize("dist,temperature", [(cb.DIST_MSE_LOGITS, 1.0), (cb.DIST_MSE_CENTRED, 1.0),
                                              (cb.DIST_KL_SOFTMAX, 1.0), (cb.DIST_KL_SOFTMAX, 2.0)])
def test_all_models_many_rows_per_cta(n, C, dtype, dist, temperature):
    models, labels, mask = rand_models(19 * n + C, ROWS, C, n, dtype)
    reduction = cb.REDUCE_SUM if temperature == 1.0 else cb.REDUCE_MEAN_VALID
    compare_all(models, labels, mask, alpha=0.8, label_smoothing=0.1, reduction=reduction, dist=dist,
                temperature=temperature)
    if dist == cb.DIST_MSE_LOGITS and n > 2:
        compare_all(models, labels, mask, alpha=0.8, peer_reduce=cb.PEERS_MEAN_TARGET, reduction=cb.REDUCE_SUM,
                    dist=dist)


@pytest.mark.parametrize("dist", [cb.DIST_MSE_LOGITS, cb.DIST_KL_SOFTMAX, cb.DIST_MSE_CENTRED])
def test_host_entry_point_with_tall_slices(dist):
    """codistill_loss_fwd_bwd_host with slices of 1500 rows (more than the CTA slots) and a ragged last
    slice: every host output against the oracle."""
    n, C, rows, chunk = 4, 9001, 3300, 1500
    models, labels, mask = rand_models(23 + dist, rows, C, n, "bf16")
    own, peers = models[0], models[1:]
    h = [torch.from_numpy(m.view(np.int16)).pin_memory() for m in models]
    h_labels, h_mask = torch.from_numpy(labels).pin_memory(), torch.from_numpy(mask).pin_memory()
    h_grad = torch.zeros((rows, C), dtype=torch.int16).pin_memory()
    h_row = torch.zeros(rows, dtype=torch.float32).pin_memory()
    h_loss = torch.zeros(1, dtype=torch.float32).pin_memory()
    h_cnt = torch.zeros(3 + n - 1, dtype=torch.int64).pin_memory()
    h_st = torch.zeros(1, dtype=torch.int32).pin_memory()
    ws = torch.empty(cb.host_workspace_bytes(n, rows, C, cb.BF16, chunk), dtype=torch.uint8, device="cuda")
    ptrs = (ctypes.c_void_p * (n - 1))(*[t.data_ptr() for t in h[1:]])
    p = cb.Params()
    p.struct_bytes = ctypes.sizeof(cb.Params)
    p.logits, p.peer_logits = h[0].data_ptr(), ctypes.cast(ptrs, ctypes.POINTER(ctypes.c_void_p))
    p.labels, p.mask = h_labels.data_ptr(), h_mask.data_ptr()
    p.n, p.dtype, p.rows, p.classes, p.row_stride = n, cb.BF16, rows, C, C
    p.alpha, p.temperature, p.label_smoothing = 0.9, 1.5, 0.05
    p.dist_kind, p.peer_reduce, p.reduction = dist, cb.PEERS_PAIRWISE_MEAN, cb.REDUCE_SUM
    p.row_loss, p.reduced_loss, p.grad_logits = h_row.data_ptr(), h_loss.data_ptr(), h_grad.data_ptr()
    p.counters, p.dev_status = h_cnt.data_ptr(), h_st.data_ptr()
    p.workspace, p.workspace_bytes = ws.data_ptr(), ws.numel()
    cb.codistill_loss_fwd_bwd_host(p, chunk)
    ref = oracle.codistill(own, peers, labels, mask, alpha=0.9, temperature=1.5, label_smoothing=0.05, dist=dist,
                           reduction=oracle.REDUCE_SUM)
    tol = TOL["bf16"]
    assert int(h_st.item()) == ref.status
    assert h_cnt.tolist() == ref.counters.tolist()
    assert abs(h_loss.item() - ref.loss) <= tol["loss_rel"] * abs(ref.loss)
    np.testing.assert_allclose(h_row.numpy().astype(np.float64), ref.row_loss, rtol=tol["loss_rel"], atol=tol["loss_floor"])
    g = synth.bf16_bits_to_f32(h_grad.numpy().view(np.uint16)).astype(np.float64)
    err = np.abs(g - ref.grad)
    assert np.all(err <= np.maximum(tol["grad_abs"], 0.75 * bf16_ulp(ref.grad))), float(err.max())
