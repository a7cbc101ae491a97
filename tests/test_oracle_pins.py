"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU needed).

Each test would fail for a plausible slip somewhere in the oracle: a dropped term, a wrong
sign, a missing 1/(n-1) or 1/C, a transposed pair of operands, a wrong tie-break.
"""
import itertools
import math
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2010_02838_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
DISTS = [oracle.DIST_MSE, oracle.DIST_KL, oracle.DIST_MSE_CENTRED, oracle.DIST_KL_REVERSE, oracle.DIST_KL_SYMMETRIC]
SHIFT_INVARIANT = (oracle.DIST_KL, oracle.DIST_MSE_CENTRED, oracle.DIST_KL_REVERSE, oracle.DIST_KL_SYMMETRIC)
PEER_REDUCES = [oracle.PEERS_PAIRWISE, oracle.PEERS_MEAN_TARGET]


def rng_inputs(seed, rows, C, n, scale=2.0, dtype=np.float32):
    g = np.random.default_rng(seed)
    own = (scale * g.standard_normal((rows, C))).astype(np.float32)
    peers = [(scale * g.standard_normal((rows, C))).astype(np.float32) for _ in range(n - 1)]
    labels = g.integers(0, C, rows).astype(np.int32)
    if dtype == np.uint16:
        own = synth.f32_to_bf16_bits(own)
        peers = [synth.f32_to_bf16_bits(p) for p in peers]
    return own, peers, labels


def widen(a):
    return a.astype(np.float64) if a.dtype == np.float32 else synth.bf16_bits_to_f32(a).astype(np.float64)


# ---------------------------------------------------------------- golden fixtures (paper-derived)
def test_hand_example_algorithm1_mse():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "hand_example_alg1_mse.txt")) if l.strip() and l[0] != "#"]
    own = np.array([[0.0, 0.0]], dtype=np.float32)
    peer = np.array([[1.0, -1.0]], dtype=np.float32)
    for alpha, loss, g0, g1 in [[float(v) for v in r] for r in rows]:
        res = oracle.codistill(own, [peer], np.array([0], np.int32), alpha=alpha, reduction=oracle.REDUCE_SUM)
        assert res.loss == pytest.approx(loss, abs=1e-15)
        assert res.grad[0] == pytest.approx([g0, g1], abs=1e-15)


def test_prediction_row_bits_section3():
    c, bits, b_pred = [int(v) for v in [l for l in open(os.path.join(GOLDEN, "prediction_bits_section3.txt"))
                                        if l.strip() and l[0] != "#"][0].split()]
    w = synth.WORKLOADS[2]
    assert w.classes == c and w.elem_bytes * 8 == bits and w.classes * w.elem_bytes * 8 == b_pred
    assert w.algorithmic_bytes() == 3 * 256 * 1000 * 4 + 9 * 256 == 3074304


# ---------------------------------------------------------------- closed forms
@pytest.mark.parametrize("dist", DISTS)
@pytest.mark.parametrize("pr", PEER_REDUCES)
@pytest.mark.parametrize("eps", [0.0, 0.1])
@pytest.mark.parametrize("T", [1.0, 2.5])
def test_all_equal_logits_give_log_C(dist, pr, eps, T):
    C, rows, n = 7, 3, 3
    own = np.full((rows, C), 1.25, dtype=np.float32)
    peers = [own.copy() for _ in range(n - 1)]
    labels = np.array([0, 3, 6], np.int32)
    res = oracle.codistill(own, peers, labels, alpha=0.7, temperature=T, label_smoothing=eps, dist=dist,
                           peer_reduce=pr, reduction=oracle.REDUCE_SUM)
    assert res.row_loss == pytest.approx(np.full(rows, math.log(C)), abs=1e-14)
    q = np.full((rows, C), eps / C)
    q[np.arange(rows), labels] += 1 - eps
    assert res.grad == pytest.approx(1.0 / C - q, abs=1e-14)


@pytest.mark.parametrize("dist", DISTS)
@pytest.mark.parametrize("pr", PEER_REDUCES)
def test_peer_equal_to_own_has_no_distillation_effect(dist, pr):
    own, _, labels = rng_inputs(1, 5, 11, 1)
    with_peers = oracle.codistill(own, [own.copy(), own.copy()], labels, alpha=3.0, temperature=1.7, dist=dist,
                                  peer_reduce=pr, reduction=oracle.REDUCE_SUM)
    alone = oracle.codistill(own, [], labels, reduction=oracle.REDUCE_SUM)
    assert with_peers.row_loss == pytest.approx(alone.row_loss, abs=1e-13)
    assert with_peers.grad == pytest.approx(alone.grad, abs=1e-13)


def test_cross_entropy_alone_is_textbook():
    own, _, labels = rng_inputs(2, 6, 9, 1)
    z = widen(own)
    res = oracle.codistill(own, [], labels, reduction=oracle.REDUCE_SUM)
    p = np.exp(z) / np.exp(z).sum(1, keepdims=True)
    assert res.row_loss == pytest.approx(-np.log(p[np.arange(6), labels]), rel=1e-13)
    onehot = np.eye(9)[labels]
    assert res.grad == pytest.approx(p - onehot, abs=1e-14)
    assert res.grad.sum(1) == pytest.approx(np.zeros(6), abs=1e-14)
    # alpha = 0 with peers present is the same thing (term omitted), as is n = 1
    _, peers, _ = rng_inputs(3, 6, 9, 3)
    res0 = oracle.codistill(own, peers, labels, alpha=0.0, reduction=oracle.REDUCE_SUM)
    assert np.array_equal(res0.row_loss, res.row_loss) and np.array_equal(res0.grad, res.grad)


@pytest.mark.parametrize("dist", DISTS)
def test_gradient_row_sums(dist):
    own, peers, labels = rng_inputs(4, 4, 13, 4)
    alpha, C = 0.9, 13
    res = oracle.codistill(own, peers, labels, alpha=alpha, temperature=1.5, label_smoothing=0.2, dist=dist,
                           reduction=oracle.REDUCE_SUM)
    if dist in SHIFT_INVARIANT:   # shift-invariant distances: their gradient sums to zero
        assert res.grad.sum(1) == pytest.approx(np.zeros(4), abs=1e-13)
    else:
        zbar = sum(widen(p) for p in peers) / 3
        expect = (2 * alpha / C) * (widen(own) - zbar).sum(1)
        assert res.grad.sum(1) == pytest.approx(expect, abs=1e-13)


@pytest.mark.parametrize("n", [3, 4, 8])
def test_mse_pairwise_vs_mean_target_identity(n):
    # 1/(n-1) sum_j |z - z_j|^2 = |z - zbar|^2 + 1/(n-1) sum_j |z_j - zbar|^2 ; gradients coincide
    own, peers, labels = rng_inputs(10 + n, 5, 17, n)
    kw = dict(alpha=1.3, reduction=oracle.REDUCE_SUM)
    a = oracle.codistill(own, peers, labels, peer_reduce=oracle.PEERS_PAIRWISE, **kw)
    b = oracle.codistill(own, peers, labels, peer_reduce=oracle.PEERS_MEAN_TARGET, **kw)
    zs = np.stack([widen(p) for p in peers])
    spread = ((zs - zs.mean(0)) ** 2).mean(axis=(0, 2))  # 1/(n-1) sum_j 1/C sum_c
    assert a.row_loss - b.row_loss == pytest.approx(1.3 * spread, rel=1e-11)
    assert a.grad == pytest.approx(b.grad, abs=1e-14)
    own2, peers2, labels2 = rng_inputs(20, 5, 17, 2)  # n = 2: everything coincides
    a2 = oracle.codistill(own2, peers2, labels2, peer_reduce=oracle.PEERS_PAIRWISE, **kw)
    b2 = oracle.codistill(own2, peers2, labels2, peer_reduce=oracle.PEERS_MEAN_TARGET, **kw)
    assert a2.row_loss == pytest.approx(b2.row_loss, rel=1e-14) and a2.grad == pytest.approx(b2.grad, abs=1e-15)


@pytest.mark.parametrize("dist", DISTS)
def test_linear_in_alpha(dist):
    own, peers, labels = rng_inputs(5, 4, 6, 3)
    f = lambda a: oracle.codistill(own, peers, labels, alpha=a, temperature=0.8, dist=dist, reduction=oracle.REDUCE_SUM)
    r0, r1, r3 = f(0.0), f(1.0), f(3.0)
    assert r3.row_loss == pytest.approx(r0.row_loss + 3 * (r1.row_loss - r0.row_loss), rel=1e-12)
    assert r3.grad == pytest.approx(r0.grad + 3 * (r1.grad - r0.grad), abs=1e-13)


def test_shift_behaviour_mse_and_kl():
    own, peers, labels = rng_inputs(6, 3, 8, 3, dtype=np.float32)
    k = 0.75  # exactly representable; keeps shifted fp32 inputs close to exact
    to64 = lambda a: a.astype(np.float64)
    # the oracle takes fp32 inputs, so build shifted inputs that are exact in fp32
    own = np.round(own * 64) / 64
    peers = [np.round(p * 64) / 64 for p in peers]
    own_s, peers_s = (own + k).astype(np.float32), [(p + k).astype(np.float32) for p in peers]
    for dist in DISTS:
        base = oracle.codistill(own, peers, labels, alpha=1.1, dist=dist, reduction=oracle.REDUCE_SUM)
        both = oracle.codistill(own_s, peers_s, labels, alpha=1.1, dist=dist, reduction=oracle.REDUCE_SUM)
        assert both.row_loss == pytest.approx(base.row_loss, rel=1e-12)
        assert both.grad == pytest.approx(base.grad, abs=1e-13)
        only_own = oracle.codistill(own_s, peers, labels, alpha=1.1, dist=dist, reduction=oracle.REDUCE_SUM)
        if dist in SHIFT_INVARIANT:   # centring removes a shift of the own logits
            assert only_own.row_loss == pytest.approx(base.row_loss, rel=1e-12)
        else:  # un-centred MSE: D changes by 2k mean_c(z - zbar) + k^2
            zbar = sum(to64(p) for p in peers) / len(peers)
            delta = 2 * k * (to64(own) - zbar).mean(1) + k * k
            assert only_own.row_loss - base.row_loss == pytest.approx(1.1 * delta, rel=1e-11)


def test_kl_form_n2_T1_closed_form_and_one_hot_limit():
    own, peers, labels = rng_inputs(7, 4, 5, 2)
    z, zp = widen(own), widen(peers[0])
    sm = lambda v: np.exp(v - v.max(1, keepdims=True)) / np.exp(v - v.max(1, keepdims=True)).sum(1, keepdims=True)
    p, t = sm(z), sm(zp)
    alpha = 0.6
    res = oracle.codistill(own, peers, labels, alpha=alpha, dist=oracle.DIST_KL, reduction=oracle.REDUCE_SUM)
    q = np.eye(5)[labels]
    assert res.grad == pytest.approx((p - q) + alpha * (p - t), abs=1e-14)
    kl = (t * (np.log(t) - np.log(p))).sum(1)
    ce = -np.log(p[np.arange(4), labels])
    assert res.row_loss == pytest.approx(ce + alpha * kl, rel=1e-13)
    # a near-one-hot peer turns the KL term into the cross-entropy against the peer's arg-max
    sharp = np.zeros((4, 5), np.float32)
    cls = np.array([1, 4, 0, 2])
    sharp[np.arange(4), cls] = 80.0
    res2 = oracle.codistill(own, [sharp], labels, alpha=1.0, dist=oracle.DIST_KL, reduction=oracle.REDUCE_SUM)
    assert res2.row_loss - ce == pytest.approx(-np.log(p[np.arange(4), cls]), rel=1e-12)


@pytest.mark.parametrize("T", [1.0, 2.5])
def test_kl_directions_swap_and_average(T):
    """The reverse direction with own and peer exchanged is the forward direction (same number), and the
    symmetric form is the average of the two; the reverse gradient is T p ((log p - log t) - KL(p || t))."""
    own, peers, labels = rng_inputs(31, 6, 11, 2)
    kw = dict(alpha=1.0, temperature=T, reduction=oracle.REDUCE_SUM)
    ce_own = oracle.codistill(own, [], labels, reduction=oracle.REDUCE_SUM).row_loss
    ce_peer = oracle.codistill(peers[0], [], labels, reduction=oracle.REDUCE_SUM).row_loss
    fwd = oracle.codistill(own, peers, labels, dist=oracle.DIST_KL, **kw)
    rev = oracle.codistill(own, peers, labels, dist=oracle.DIST_KL_REVERSE, **kw)
    sym = oracle.codistill(own, peers, labels, dist=oracle.DIST_KL_SYMMETRIC, **kw)
    fwd_swapped = oracle.codistill(peers[0], [own], labels, dist=oracle.DIST_KL, **kw)
    assert rev.row_loss - ce_own == pytest.approx(fwd_swapped.row_loss - ce_peer, rel=1e-12, abs=1e-14)
    assert sym.row_loss == pytest.approx(0.5 * (fwd.row_loss + rev.row_loss), rel=1e-13)
    assert sym.grad == pytest.approx(0.5 * (fwd.grad + rev.grad), abs=1e-14)
    # the closed form of the reverse gradient, written out with numpy
    z, v = widen(own) / T, widen(peers[0]) / T
    lp = z - np.log(np.exp(z - z.max(1, keepdims=True)).sum(1, keepdims=True)) - z.max(1, keepdims=True)
    lt = v - np.log(np.exp(v - v.max(1, keepdims=True)).sum(1, keepdims=True)) - v.max(1, keepdims=True)
    p = np.exp(lp)
    kl = (p * (lp - lt)).sum(1, keepdims=True)
    ce_grad = oracle.codistill(own, [], labels, reduction=oracle.REDUCE_SUM).grad
    assert rev.grad - ce_grad == pytest.approx(T * p * ((lp - lt) - kl), abs=1e-13)
    assert rev.row_loss - ce_own == pytest.approx(T * T * kl[:, 0], rel=1e-12)
    assert np.all(rev.row_loss - ce_own >= 0) and np.all(fwd.row_loss - ce_own >= 0)    # a divergence is never negative


def test_kl_temperature_scaling():
    # D_T(z, z') = T^2 * D_1(z/T, z'/T); use power-of-two T so z/T is exact in fp32
    own, peers, labels = rng_inputs(8, 3, 6, 3)
    T = 2.0
    for pr in PEER_REDUCES:
        a0 = oracle.codistill(own, peers, labels, alpha=0.0, reduction=oracle.REDUCE_SUM)
        a = oracle.codistill(own, peers, labels, alpha=1.0, temperature=T, dist=oracle.DIST_KL, peer_reduce=pr,
                             reduction=oracle.REDUCE_SUM)
        b0 = oracle.codistill(own / T, [p / T for p in peers], labels, alpha=0.0, reduction=oracle.REDUCE_SUM)
        b = oracle.codistill(own / T, [p / T for p in peers], labels, alpha=1.0, temperature=1.0,
                             dist=oracle.DIST_KL, peer_reduce=pr, reduction=oracle.REDUCE_SUM)
        assert a.row_loss - a0.row_loss == pytest.approx(T * T * (b.row_loss - b0.row_loss), rel=1e-11)
        assert a.grad - a0.grad == pytest.approx(T * (b.grad - b0.grad), abs=1e-13)  # d/dz = (1/T) d/d(z/T)


# ---------------------------------------------------------------- label smoothing, mask, reductions
def test_label_smoothing_decomposition():
    own, _, labels = rng_inputs(9, 5, 12, 1)
    eps, C = 0.3, 12
    z = widen(own)
    logp = z - np.log(np.exp(z).sum(1, keepdims=True))
    res = oracle.codistill(own, [], labels, label_smoothing=eps, reduction=oracle.REDUCE_SUM)
    expect = -(1 - eps) * logp[np.arange(5), labels] - (eps / C) * logp.sum(1)
    assert res.row_loss == pytest.approx(expect, rel=1e-13)


def test_mask_bad_labels_and_reductions():
    own, peers, labels = rng_inputs(11, 8, 6, 3)
    mask = np.array([1, 0, 1, 1, 0, 1, 1, 1], np.uint8)
    labels = labels.copy()
    labels[2] = 6    # == classes: not a class id
    labels[5] = -1
    res = oracle.codistill(own, peers, labels, mask, alpha=0.4, reduction=oracle.REDUCE_MEAN_VALID)
    keep = np.array([0, 3, 6, 7])
    ref = oracle.codistill(own[keep], [p[keep] for p in peers], labels[keep], None, alpha=0.4,
                           reduction=oracle.REDUCE_SUM)
    assert res.status == 1 and ref.status == 0
    assert list(res.counters[:2]) == [4, 4] and res.counters[2:].tolist() == ref.counters[2:].tolist()
    assert res.loss == pytest.approx(ref.loss / 4, rel=1e-14)
    assert res.grad[keep] == pytest.approx(ref.grad / 4, abs=1e-15)
    drop = np.array([1, 2, 4, 5])
    assert np.all(res.grad[drop] == 0) and np.all(res.row_loss[drop] == 0)
    # all rows masked: loss 0 (division by max(n_valid, 1)), not NaN
    none = oracle.codistill(own, peers, labels, np.zeros(8, np.uint8), alpha=0.4)
    assert none.loss == 0.0 and np.all(none.grad == 0) and list(none.counters[:3]) == [0, 8, 0]
    # zero rows
    empty = oracle.codistill(own[:0], [p[:0] for p in peers], labels[:0])
    assert empty.loss == 0.0 and empty.counters.tolist() == [0, 0, 0, 0, 0]


def test_row_stride_and_grad_row_range():
    own, peers, labels = rng_inputs(12, 6, 10, 2)
    pad = lambda a: np.ascontiguousarray(np.concatenate([a, np.full((6, 3), 99.0, np.float32)], axis=1))
    a = oracle.codistill(own, peers, labels, alpha=0.5)
    b = oracle.codistill(pad(own), [pad(p) for p in peers], labels, classes=10, alpha=0.5, grad_rows=(2, 5))
    assert b.loss == a.loss and np.array_equal(b.grad, a.grad[2:5])


def test_bf16_inputs_are_widened_exactly():
    own, peers, labels = rng_inputs(13, 4, 9, 3, dtype=np.uint16)
    a = oracle.codistill(own, peers, labels, alpha=0.8)
    b = oracle.codistill(synth.bf16_bits_to_f32(own), [synth.bf16_bits_to_f32(p) for p in peers], labels, alpha=0.8)
    assert a.loss == b.loss and np.array_equal(a.grad, b.grad)


# ---------------------------------------------------------------- counters: brute force with planted ties
def test_counters_brute_force_with_ties():
    g = np.random.default_rng(14)
    rows, C, n = 40, 5, 4
    own = g.integers(-2, 3, (rows, C)).astype(np.float32)      # few distinct values: many ties
    peers = [g.integers(-2, 3, (rows, C)).astype(np.float32) for _ in range(n - 1)]
    own[0, :] = 0.0
    own[0, 2] = -0.0                                             # -0.0 ties with +0.0: index 0 wins
    labels = g.integers(0, C, rows).astype(np.int32)
    mask = (g.random(rows) > 0.2).astype(np.uint8)
    res = oracle.codistill(own, peers, labels, mask)

    def first_argmax(v):
        best = 0
        for c in range(1, len(v)):
            if v[c] > v[best]:
                best = c
        return best

    nv = nm = nc = 0
    agree = [0] * (n - 1)
    for r in range(rows):
        if not mask[r]:
            nm += 1
            continue
        nv += 1
        a = first_argmax(own[r])
        nc += int(a == labels[r])
        for j in range(n - 1):
            agree[j] += int(first_argmax(peers[j][r]) == a)
    assert res.counters.tolist() == [nv, nm, nc] + agree


# ---------------------------------------------------------------- finite differences and autograd
def _scalar_loss(own64, peers, labels, mask, kw):
    return oracle.codistill(own64.astype(np.float32), peers, labels, mask, want_grad=False, **kw).loss


@pytest.mark.parametrize("dist,pr,eps,T,use_mask,red", [
    c for c in itertools.product(DISTS, PEER_REDUCES, [0.0, 0.15], [1.0, 2.0], [False, True],
                                 [oracle.REDUCE_SUM, oracle.REDUCE_MEAN_VALID])])
def test_central_finite_differences(dist, pr, eps, T, use_mask, red):
    rows, C, n = 3, 7, 4
    g = np.random.default_rng(15)
    # inputs on a 2^-6 grid so that +-h with h = 2^-10 stays exact in fp32
    own = (np.round(g.standard_normal((rows, C)) * 64) / 64).astype(np.float32)
    peers = [(np.round(g.standard_normal((rows, C)) * 64) / 64).astype(np.float32) for _ in range(n - 1)]
    labels = g.integers(0, C, rows).astype(np.int32)
    mask = np.array([1, 0, 1], np.uint8) if use_mask else None
    kw = dict(alpha=0.7, temperature=T, label_smoothing=eps, dist=dist, peer_reduce=pr, reduction=red)
    res = oracle.codistill(own, peers, labels, mask, **kw)
    h = 2.0 ** -10
    num = np.zeros((rows, C))
    for r in range(rows):
        for c in range(C):
            up, dn = own.copy(), own.copy()
            up[r, c] += h
            dn[r, c] -= h
            # Richardson-extrapolated central difference (error O(h^4))
            up2, dn2 = own.copy(), own.copy()
            up2[r, c] += 2 * h
            dn2[r, c] -= 2 * h
            d1 = (_scalar_loss(up, peers, labels, mask, kw) - _scalar_loss(dn, peers, labels, mask, kw)) / (2 * h)
            d2 = (_scalar_loss(up2, peers, labels, mask, kw) - _scalar_loss(dn2, peers, labels, mask, kw)) / (4 * h)
            num[r, c] = (4 * d1 - d2) / 3
    assert res.grad == pytest.approx(num, abs=2e-9)


def _torch_reference(own, peers, labels, mask, alpha, T, eps, dist, pr, red):
    """The same scalar composed from torch CPU float64 library ops + autograd (the paper's
    experiments were written in PyTorch): cross_entropy with label smoothing, mse_loss, kl_div."""
    F = torch.nn.functional
    z = torch.tensor(widen(own), dtype=torch.float64, requires_grad=True)
    ps = [torch.tensor(widen(p), dtype=torch.float64) for p in peers]
    y = torch.tensor(labels, dtype=torch.long)
    valid = torch.ones(len(labels), dtype=torch.bool) if mask is None else torch.tensor(mask.astype(bool))
    ce = F.cross_entropy(z, y, reduction="none", label_smoothing=eps)
    if ps and alpha != 0:
        if pr == oracle.PEERS_MEAN_TARGET:
            ps = [torch.stack(ps).mean(0)]
        ds = []
        for p in ps:
            if dist == oracle.DIST_MSE:
                ds.append(F.mse_loss(z, p, reduction="none").mean(1))
            elif dist == oracle.DIST_MSE_CENTRED:
                ds.append(F.mse_loss(z - z.mean(1, keepdim=True), p - p.mean(1, keepdim=True), reduction="none").mean(1))
            else:
                lp, lt = F.log_softmax(z / T, 1), F.log_softmax(p / T, 1)
                fwd = T * T * F.kl_div(lp, lt, reduction="none", log_target=True).sum(1)    # KL(t || p)
                rev = T * T * F.kl_div(lt, lp, reduction="none", log_target=True).sum(1)    # KL(p || t)
                ds.append({oracle.DIST_KL: fwd, oracle.DIST_KL_REVERSE: rev, oracle.DIST_KL_SYMMETRIC: 0.5 * (fwd + rev)}[dist])
        row = ce + alpha * torch.stack(ds).mean(0)
    else:
        row = ce
    row = torch.where(valid, row, torch.zeros_like(row))
    total = row.sum() if red == oracle.REDUCE_SUM else row.sum() / max(int(valid.sum()), 1)
    total.backward()
    return row.detach().numpy(), float(total.detach()), z.grad.numpy()


@pytest.mark.parametrize("dist", DISTS)
@pytest.mark.parametrize("pr", PEER_REDUCES)
@pytest.mark.parametrize("n,rows,C,dtype", [(2, 5, 10, np.float32), (4, 33, 257, np.uint16), (8, 7, 1000, np.float32)])
def test_against_torch_float64_autograd(dist, pr, n, rows, C, dtype):
    own, peers, labels = rng_inputs(100 + n, rows, C, n, dtype=dtype)
    mask = (np.random.default_rng(5).random(rows) > 0.25).astype(np.uint8)
    for red, eps, T, m in [(oracle.REDUCE_SUM, 0.0, 1.0, None), (oracle.REDUCE_MEAN_VALID, 0.1, 2.0, mask)]:
        res = oracle.codistill(own, peers, labels, m, alpha=0.5, temperature=T, label_smoothing=eps, dist=dist,
                               peer_reduce=pr, reduction=red)
        row, total, grad = _torch_reference(own, peers, labels, m, 0.5, T, eps, dist, pr, red)
        assert res.row_loss == pytest.approx(row, rel=1e-12, abs=1e-13)
        assert res.loss == pytest.approx(total, rel=1e-12)
        assert res.grad == pytest.approx(grad, abs=1e-13)


# ---------------------------------------------------------------- the synthetic recipe
def test_synth_is_counter_based_and_matches_recipe():
    w = synth.WORKLOADS[3]
    full = synth.make_model_logits(w, 2)
    part = synth.make_model_logits(w, 2, 100, 117)
    assert np.array_equal(full[100:117], part)
    w4 = synth.WORKLOADS[4]
    m = synth.make_mask(w4)
    assert m.shape == (8192,) and int((m == 0).sum()) == 819
    seqs = m.reshape(256, 32)
    assert np.all(np.diff(seqs.astype(int), axis=1) <= 0)          # padding only at the end of a sentence
    assert sorted(set((seqs == 0).sum(1))) == [3, 4] and int(((seqs == 0).sum(1) == 4).sum()) == 51
    m5 = synth.make_mask(synth.WORKLOADS[5])
    assert int((m5 == 0).sum()) == 819 and int(((m5.reshape(512, 32) == 0).sum(1) == 2).sum()) == 307
    x = synth.bf16_bits_to_f32(synth.make_model_logits(synth.scaled(w4, rows=64), 0))
    assert abs(float(x.std()) - 1.5) < 0.01 and abs(float(x.mean())) < 0.01
    # RNE rounding to bf16: halfway cases go to even
    halves = np.array([1.00390625, 1.01171875], np.float32)        # 1 + 2^-8, 1 + 3*2^-8
    assert synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(halves)).tolist() == [1.0, 1.015625]
    assert synth.WORKLOADS[4].algorithmic_bytes() == 1610686464
    assert synth.WORKLOADS[4].algorithmic_bytes(True) == 1503338496
    assert synth.WORKLOADS[5].algorithmic_bytes() == 14821539840


def test_all_models_loop_and_centred_identity():
    """Algorithm 1's inner loop over the n models: model i's peers are the other models in increasing
    index; and the closed form behind the all-models kernel, sum_{j != i} (z_i - z_j)^2 =
    n z'_i^2 + sum_j z'_j^2 with z' centred on the mean over the models (brute force in numpy)."""
    g = np.random.default_rng(12)
    rows, C, n, alpha = 5, 9, 4, 0.7
    models = [g.standard_normal((rows, C)).astype(np.float32) for _ in range(n)]
    labels = g.integers(0, C, rows).astype(np.int32)
    res = oracle.codistill_all(models, labels, None, alpha=alpha, reduction=oracle.REDUCE_SUM)
    assert len(res) == n
    z = np.stack([m.astype(np.float64) for m in models])           # [n, rows, C]
    zc = z - z.mean(axis=0, keepdims=True)
    q = (zc ** 2).sum(axis=0)
    for i in range(n):
        single = oracle.codistill(models[i], [models[j] for j in range(n) if j != i], labels, None, alpha=alpha,
                                  reduction=oracle.REDUCE_SUM)
        assert np.array_equal(res[i].row_loss, single.row_loss) and np.array_equal(res[i].grad, single.grad)
        ce = oracle.codistill(models[i], [], labels, None, reduction=oracle.REDUCE_SUM).row_loss
        d_closed = (n * zc[i] ** 2 + q).sum(axis=1) / ((n - 1) * C)
        np.testing.assert_allclose((res[i].row_loss - ce) / alpha, d_closed, rtol=1e-12, atol=1e-14)
        # counters: agreement with model j is equality of the first arg-maxes
        am = z.argmax(axis=2)
        others = [j for j in range(n) if j != i]
        assert res[i].counters[3:].tolist() == [int((am[i] == am[j]).sum()) for j in others]


def test_all_models_kl_shared_column_sums():
    """The closed form behind the all-models KL kernel: with t_j = softmax(z_j / T), Q = sum_j t_j and
    E = sum_j t_j log t_j per column, sum_{j != i} KL(t_j || t_i) = sum_c (E_c - Q_c log t_ic) and the
    derivative of T^2 times it with respect to z_i is T (n t_i - Q); brute force in numpy against the
    oracle's pairwise loop."""
    g = np.random.default_rng(31)
    rows, C, n, alpha, T = 4, 13, 5, 0.9, 2.5
    models = [(1.5 * g.standard_normal((rows, C))).astype(np.float32) for _ in range(n)]
    labels = g.integers(0, C, rows).astype(np.int32)
    kw = dict(alpha=alpha, temperature=T, dist=oracle.DIST_KL, reduction=oracle.REDUCE_SUM)
    res = oracle.codistill_all(models, labels, None, **kw)
    z = np.stack([m.astype(np.float64) for m in models]) / T
    log_t = z - np.log(np.exp(z).sum(axis=2, keepdims=True))
    t = np.exp(log_t)
    Q, E = t.sum(axis=0), (t * log_t).sum(axis=0)
    for i in range(n):
        plain = oracle.codistill(models[i], [], labels, None, reduction=oracle.REDUCE_SUM)
        d_closed = T * T * (E - Q * log_t[i]).sum(axis=1) / (n - 1)
        np.testing.assert_allclose((res[i].row_loss - plain.row_loss) / alpha, d_closed, rtol=1e-11, atol=1e-13)
        np.testing.assert_allclose((res[i].grad - plain.grad) / alpha, T * (n * t[i] - Q) / (n - 1), rtol=1e-11, atol=1e-13)


@pytest.mark.parametrize("pr", PEER_REDUCES)
def test_centred_mse_is_the_variance_of_the_difference(pr):
    """Appendix "Implementation Details" mentions centring the logits: with both logit vectors centred
    on their class means, D_j = var_c(z - z^(j)) = MSE_j - (mean_c (z - z^(j)))^2, and the derivative is
    (2/C) (d_c - mean_c d); brute force in numpy."""
    own, peers, labels = rng_inputs(21, 5, 11, 4)
    alpha, C, P = 0.6, 11, 3
    kw = dict(alpha=alpha, peer_reduce=pr, reduction=oracle.REDUCE_SUM)
    cen = oracle.codistill(own, peers, labels, dist=oracle.DIST_MSE_CENTRED, **kw)
    ce = oracle.codistill(own, [], labels, reduction=oracle.REDUCE_SUM)
    z = widen(own)
    if pr == oracle.PEERS_MEAN_TARGET:
        targets = [sum(widen(p) for p in peers) / P]
    else:
        targets = [widen(p) for p in peers]
    D = np.zeros(5)
    dD = np.zeros_like(z)
    for t in targets:
        d = z - t
        D += (d ** 2).mean(1) - d.mean(1) ** 2
        dD += (2.0 / C) * (d - d.mean(1, keepdims=True))
    D /= len(targets)
    dD /= len(targets)
    np.testing.assert_allclose(cen.row_loss, ce.row_loss + alpha * D, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(cen.grad, ce.grad + alpha * dD, rtol=0, atol=1e-14)
