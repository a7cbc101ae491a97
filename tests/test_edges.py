"""GPU parity on edge cases: ragged and unaligned rows, row pitch, degenerate sizes, masks,
planted arg-max ties, bad labels, optional outputs, determinism, untouched guard bands."""
import numpy as np
import pytest
import torch

import oracle
from paper_2010_02838_b200 import binding as cb
from paper_2010_02838_b200 import synth

from helpers import compare, to_device

pytestmark = pytest.mark.gpu


def rand_inputs(seed, rows, C, n, dtype, scale=1.5):
    g = np.random.default_rng(seed)
    mk = lambda: (scale * g.standard_normal((rows, C))).astype(np.float32)
    own, peers = mk(), [mk() for _ in range(n - 1)]
    labels = g.integers(0, C, rows).astype(np.int32)
    if dtype == "bf16":
        own, peers = synth.f32_to_bf16_bits(own), [synth.f32_to_bf16_bits(p) for p in peers]
    return own, peers, labels


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("C", [1, 2, 7, 33, 257, 1000, 1023, 4099, 9001, 20011])
@pytest.mark.parametrize("dist", [0, 1, 2, 3, 4])
def test_ragged_class_counts(dtype, C, dist):
    rows = 37 if C < 5000 else 11
    own, peers, labels = rand_inputs(C, rows, C, 3, dtype)
    mask = (np.arange(rows) % 5 != 1).astype(np.uint8)
    compare(own, peers, labels, mask, alpha=0.8, temperature=1.5, label_smoothing=0.05, dist=dist,
            reduction=cb.REDUCE_SUM)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("C,stride", [(10, 16), (1000, 1024), (50257, 50264), (33000, 33008), (5, 9)])
def test_row_pitch(dtype, C, stride):
    rows = 9
    own, peers, labels = rand_inputs(7, rows, stride, 2, dtype)
    plan, out, ref = compare(own, peers, labels, None, classes=C, alpha=1.0, reduction=cb.REDUCE_SUM)
    # the padding columns of the gradient are never written
    g = torch.full((rows, stride), 7.0, dtype=plan.out.grad.dtype, device="cuda")
    plan.params.grad_logits = g.data_ptr()
    plan.run()
    torch.cuda.synchronize()
    assert torch.all(g[:, C:].float() == 7.0)
    assert torch.equal(g[:, :C], out.grad)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_degenerate_shapes(dtype):
    for rows, C, n in [(1, 1, 1), (1, 5, 2), (3, 40000, 1), (2, 3, 8)]:
        own, peers, labels = rand_inputs(rows * 31 + C, rows, C, n, dtype)
        for red in (0, 1):
            compare(own, peers, labels, None, alpha=1.2, reduction=red)


def test_zero_rows_and_all_masked():
    own, peers, labels = rand_inputs(3, 6, 50, 3, "f32")
    e = cb.Plan(to_device(own[:0]), [to_device(p[:0]) for p in peers], to_device(labels[:0]))
    out = e.run()
    torch.cuda.synchronize()
    assert out.loss.item() == 0.0 and out.counters.cpu().tolist() == [0, 0, 0, 0, 0] and out.status.item() == 0
    plan, out, ref = compare(own, peers, labels, np.zeros(6, np.uint8), alpha=1.0)
    assert out.loss.item() == 0.0 and torch.all(out.grad == 0)


@pytest.mark.parametrize("dist", [0, 1, 2])
def test_alpha_zero_n1_and_peer_equal_own(dist):
    own, peers, labels = rand_inputs(4, 20, 300, 3, "bf16")
    compare(own, peers, labels, None, alpha=0.0, dist=dist, reduction=1)     # term omitted, agreement still counted
    compare(own, [], labels, None, alpha=1.0, dist=dist, reduction=1)         # n = 1
    plan, out, ref = compare(own, [own.copy(), own.copy()], labels, None, alpha=2.0, dist=dist, reduction=1)
    alone = oracle.codistill(own, [], labels, reduction=1)
    np.testing.assert_allclose(out.row_loss.cpu().numpy(), alone.row_loss, rtol=2e-3)
    assert out.counters.cpu().tolist()[3:] == [20, 20]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("C", [6, 1000, 20000, 40000])
def test_planted_argmax_ties(dtype, C):
    rows, n = 24, 4
    g = np.random.default_rng(C)
    mk = lambda: g.integers(-3, 4, (rows, C)).astype(np.float32)   # few distinct values: many ties
    own, peers = mk(), [mk() for _ in range(n - 1)]
    own[0, :] = 0.0
    own[0, C // 2] = -0.0                                           # -0.0 ties with +0.0
    peers[0][1, :] = own[1, :]                                       # a sure agreement
    top = float(own[2].max()) + 1
    own[2, [1, C - 1]] = top                                         # duplicate maximum: first index wins
    peers[1][2, :] = -5.0
    peers[1][2, C - 1] = 9.0                                         # peer picks the later duplicate: no agreement
    labels = np.array([int(np.argmax(own[r])) if r % 2 else int(g.integers(0, C)) for r in range(rows)], np.int32)
    if dtype == "bf16":
        own, peers = synth.f32_to_bf16_bits(own), [synth.f32_to_bf16_bits(p) for p in peers]
    compare(own, peers, labels, None, alpha=0.01, reduction=1, check_ulp=False)


def test_bad_labels_set_status_and_mask_the_row():
    own, peers, labels = rand_inputs(5, 40, 1000, 2, "f32")
    labels = labels.copy()
    labels[3], labels[17], labels[39] = 1000, -1, 2 ** 30
    mask = np.ones(40, np.uint8)
    mask[17] = 0                                                     # masked rows may carry any label
    plan, out, ref = compare(own, peers, labels, mask, alpha=1.0)
    assert out.status.item() == cb.DEV_BAD_LABEL and out.counters.cpu().tolist()[:2] == [37, 3]
    assert torch.all(out.grad[[3, 17, 39]] == 0)


def test_optional_outputs_and_forward_only():
    own, peers, labels = rand_inputs(6, 50, 777, 2, "bf16")
    args = (to_device(own), [to_device(p) for p in peers], to_device(labels))
    full = cb.Plan(*args, reduction=1).run()
    fwd = cb.Plan(*args, reduction=1, want_grad=False, want_row_loss=False, want_counters=False).run()
    torch.cuda.synchronize()
    assert fwd.grad is None and fwd.row_loss is None and fwd.counters is None
    assert fwd.loss.item() == full.loss.item()


@pytest.mark.parametrize("shape", [(64, 10, "f32"), (200, 1000, "bf16"), (48, 32768, "bf16"), (40, 50257, "bf16")])
def test_determinism_and_guard_bands(shape):
    rows, C, dtype = shape
    own, peers, labels = rand_inputs(8, rows, C, 3, dtype)
    mask = (np.arange(rows) % 9 != 2).astype(np.uint8)
    d_own, d_peers = to_device(own), [to_device(p) for p in peers]
    guard = 64
    buf = torch.full((rows * C + 2 * guard,), 3.0, dtype=d_own.dtype, device="cuda")
    rl = torch.full((rows + 2 * guard,), 5.0, dtype=torch.float32, device="cuda")
    runs = []
    for _ in range(2):
        plan = cb.Plan(d_own, d_peers, to_device(labels), to_device(mask), alpha=0.9)
        plan.params.grad_logits = buf.data_ptr() + guard * buf.element_size()
        plan.params.row_loss = rl.data_ptr() + guard * 4
        out = plan.run()
        torch.cuda.synchronize()
        runs.append((buf.clone(), rl.clone(), out.loss.clone(), out.counters.clone()))
    for a, b in zip(runs[0], runs[1]):
        assert torch.equal(a, b)                                      # run-to-run bit identity
    assert torch.all(buf[:guard].float() == 3.0) and torch.all(buf[-guard:].float() == 3.0)
    assert torch.all(rl[:guard] == 5.0) and torch.all(rl[-guard:] == 5.0)
    ref = oracle.codistill(own, peers, labels, mask, alpha=0.9)
    g = buf[guard:-guard].view(rows, C).double().cpu().numpy()
    assert np.abs(g - ref.grad).max() <= (1e-6 if dtype == "f32" else 2e-3)


@pytest.mark.parametrize("regime,dist", [("tma", 0), ("stream", 0), ("stream", 1)])
def test_host_buffer_entry_point(monkeypatch, regime, dist):
    """codistill_loss_fwd_bwd_host: host pointers in, host results out, several slices (each slice is a
    launch on a row range: served by either long-row kernel, and by the KL kernel)."""
    import ctypes
    monkeypatch.setenv("CODISTILL_REGIME", regime)
    w = synth.scaled(synth.WORKLOADS[4], rows=96, classes=4096)
    own, peers, labels, mask = synth.make_inputs(w)
    n, rows, C = w.n, w.rows, w.classes
    pin = lambda a: torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).pin_memory()
    h_own, h_peers, h_labels, h_mask = pin(own), [pin(p) for p in peers], pin(labels), pin(mask)
    h_grad = torch.empty_like(h_own).pin_memory()
    h_row = torch.empty(rows, dtype=torch.float32).pin_memory()
    h_loss = torch.empty(1, dtype=torch.float32).pin_memory()
    h_cnt = torch.empty(3 + n - 1, dtype=torch.int64).pin_memory()
    h_st = torch.empty(1, dtype=torch.int32).pin_memory()
    chunk = 40
    ws = torch.empty(cb.host_workspace_bytes(n, rows, C, cb.BF16, chunk), dtype=torch.uint8, device="cuda")
    ptrs = (ctypes.c_void_p * 1)(h_peers[0].data_ptr())
    p = cb.Params()
    p.struct_bytes = ctypes.sizeof(cb.Params)
    p.logits, p.peer_logits = h_own.data_ptr(), ctypes.cast(ptrs, ctypes.POINTER(ctypes.c_void_p))
    p.labels, p.mask = h_labels.data_ptr(), h_mask.data_ptr()
    p.n, p.dtype, p.rows, p.classes, p.row_stride = n, cb.BF16, rows, C, C
    p.alpha, p.temperature, p.label_smoothing = 1.0, 1.0, 0.1
    p.dist_kind = dist
    p.row_loss, p.reduced_loss, p.grad_logits = h_row.data_ptr(), h_loss.data_ptr(), h_grad.data_ptr()
    p.counters, p.dev_status = h_cnt.data_ptr(), h_st.data_ptr()
    p.workspace, p.workspace_bytes = ws.data_ptr(), ws.numel()
    cb.codistill_loss_fwd_bwd_host(p, chunk)
    ref = oracle.codistill(own, peers, labels, mask, alpha=1.0, label_smoothing=0.1, dist=dist)
    assert abs(h_loss.item() - ref.loss) <= 2e-3 * abs(ref.loss)
    assert h_cnt.tolist() == ref.counters.tolist() and h_st.item() == 0
    np.testing.assert_allclose(h_row.numpy(), ref.row_loss, rtol=2e-3)
    g = synth.bf16_bits_to_f32(h_grad.numpy().view(np.uint16)).astype(np.float64)
    assert np.abs(g - ref.grad).max() <= 2e-3


def test_expired_wait_sets_the_status_bit_and_the_context_stays_usable():
    """A wait on an asynchronous copy that runs out of time ends in CODISTILL_DEV_TIMEOUT and a normal
    kernel exit.  The diagnostic call waits 1 ms on a barrier nothing completes (no copy is involved);
    an ordinary call right after it gives the oracle's result."""
    status = cb.selftest_bounded_wait(1_000_000)
    torch.cuda.synchronize()
    assert int(status.item()) == cb.DEV_TIMEOUT
    own, peers, labels = rand_inputs(3, 12, 8192, 2, "bf16")
    compare(own, peers, labels, None, alpha=1.0, reduction=cb.REDUCE_SUM, expect_regime="tma")
    with pytest.raises(cb.CodistillError):
        cb.selftest_bounded_wait(10 ** 9)     # limits beyond 100 ms are refused on the host


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("C,n", [(1, 2), (10, 2), (33, 4), (257, 8), (1000, 3), (1024, 8), (1023, 1)])
def test_single_launch_short_row_kernel(dtype, C, n):
    """Short rows in one cooperative launch: every lane count per row, ragged last packets, a mask with a bad
    label, planted arg-max ties, both reductions, guard bands around the gradient, two identical runs."""
    rows = 77
    own, peers, labels = rand_inputs(5 * C + n, rows, C, n, dtype, scale=2.0)
    mask = (np.arange(rows) % 6 != 4).astype(np.uint8)
    labels[3] = C + 5                      # a label that is not a class: the row counts as masked, status bit raised
    if C > 4:
        for r in range(0, rows, 5):        # equal maxima in own and peers: the first one decides
            own[r, [1, C - 2]] = own[r].max() + 1
            for p in peers:
                p[r, [C - 2]] = p[r].max() + 1
    for pr, red in ((cb.PEERS_PAIRWISE_MEAN, cb.REDUCE_SUM), (cb.PEERS_MEAN_TARGET, cb.REDUCE_MEAN_VALID)):
        plan, out, ref = compare(own, peers, labels, mask, alpha=0.8, label_smoothing=0.1, peer_reduce=pr, reduction=red,
                                 expect_regime="short")
        assert int(out.status.item()) == cb.DEV_BAD_LABEL
    g = torch.full((rows * C + 64,), 3.0, dtype=plan.out.grad.dtype, device="cuda")
    plan.params.grad_logits = g[32:].data_ptr()
    first = (out.grad.clone(), out.row_loss.clone(), out.loss.clone(), out.counters.clone())
    plan.run()
    torch.cuda.synchronize()
    assert torch.all(g[:32].float() == 3.0) and torch.all(g[32 + rows * C:].float() == 3.0)
    assert torch.equal(g[32:32 + rows * C].view(rows, C), first[0])
    assert torch.equal(first[1], out.row_loss) and torch.equal(first[2], out.loss) and torch.equal(first[3], out.counters)
