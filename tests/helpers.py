"""Shared helpers of the GPU parity tests: move seeded numpy inputs to the device, run the CUDA
library through its C ABI (via the ctypes binding) and the CPU oracle on the same bits, compare."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2010_02838_b200 import binding as cb
from paper_2010_02838_b200 import synth

# tolerances of the objective: fp32 logits / bf16 logits with fp32 accumulation.  loss_floor is an
# absolute floor for losses that are exactly zero in exact arithmetic (C = 1, identical peers): a few
# fp32 roundings of O(1) terms.
TOL = {
    "f32": dict(loss_rel=1e-5, loss_floor=2e-7, grad_abs=1e-6),
    "bf16": dict(loss_rel=2e-3, loss_floor=2e-7, grad_abs=2e-3),
}


def to_device(a: np.ndarray | None) -> torch.Tensor | None:
    if a is None:
        return None
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(a).cuda()


def grad_to_f64(g: torch.Tensor) -> np.ndarray:
    return g.detach().to(torch.float64).cpu().numpy()


def bf16_round(x: np.ndarray) -> np.ndarray:
    return synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(x.astype(np.float32))).astype(np.float64)


def bf16_ulp(x: np.ndarray) -> np.ndarray:
    """Spacing of bf16 numbers around |x| (8 significant bits)."""
    ax = np.maximum(np.abs(x), 2.0 ** -126)
    return 2.0 ** (np.floor(np.log2(ax)) - 7)


def run_gpu(own, peers, labels, mask, *, classes=None, **opt):
    """Returns (Outputs on host as numpy, regime)."""
    d_own, d_peers = to_device(own), [to_device(p) for p in peers]
    if classes is not None and classes != own.shape[1]:
        d_own_v, d_peers_v = d_own[:, :classes], [p[:, :classes] for p in d_peers]
    else:
        d_own_v, d_peers_v = d_own, d_peers
    plan = cb.Plan(d_own_v, d_peers_v, to_device(labels), to_device(mask), classes=classes, **opt)
    out = plan.run()
    torch.cuda.synchronize()
    return plan, out


def compare(own, peers, labels, mask, *, classes=None, alpha=1.0, temperature=1.0, label_smoothing=0.0,
            dist=0, peer_reduce=0, reduction=0, expect_regime=None, check_ulp=True):
    """Run both sides on the same inputs and assert parity; returns the GPU plan."""
    kind = "f32" if own.dtype == np.float32 else "bf16"
    tol = TOL[kind]
    C = own.shape[1] if classes is None else classes
    opt = dict(alpha=alpha, temperature=temperature, label_smoothing=label_smoothing, dist=dist,
               peer_reduce=peer_reduce, reduction=reduction)
    plan, out = run_gpu(own, peers, labels, mask, classes=classes, **opt)
    if expect_regime is not None:
        assert plan.regime == expect_regime, (plan.regime, expect_regime)
    ref = oracle.codistill(own, peers, labels, mask, classes=classes, **opt)

    assert int(out.status.item()) == ref.status
    assert out.counters.cpu().numpy().tolist() == ref.counters.tolist()           # integers: bit-exact
    loss = float(out.loss.item())
    assert abs(loss - ref.loss) <= tol["loss_rel"] * abs(ref.loss) + tol["loss_floor"], (loss, ref.loss)
    row = out.row_loss.cpu().numpy().astype(np.float64)
    np.testing.assert_allclose(row, ref.row_loss, rtol=tol["loss_rel"], atol=tol["loss_floor"])
    g = grad_to_f64(out.grad)[:, :C]
    err = np.abs(g - ref.grad)
    if kind == "f32":
        if dist in (cb.DIST_KL_REVERSE, cb.DIST_KL_SYMMETRIC):
            # the reverse direction's gradient T p ((log p - log t) - KL) is not bounded by 1 like the other forms',
            # and it is a difference of log-ratios of size L = 2 max|logit| / T + log C, each of which fp32 holds to
            # L 2^-24: a few such roundings bound the absolute error; beyond 1 the tolerance becomes relative
            widest = max(float(np.abs(a).max()) for a in [own] + list(peers)) if len(peers) else 0.0
            L = 2.0 * widest / temperature + np.log(C)
            extra = 4 * 2.0 ** -24 * abs(alpha) * temperature * L
            assert np.all(err <= tol["grad_abs"] * np.maximum(1.0, np.abs(ref.grad)) + extra), float(err.max())
        else:
            assert err.max(initial=0.0) <= tol["grad_abs"], err.max()
    else:
        # |g| <= 1: the stated absolute tolerance; larger values are bounded by bf16 rounding itself
        bound = np.maximum(tol["grad_abs"], 0.75 * bf16_ulp(ref.grad))
        assert np.all(err <= bound), float((err - bound).max())
        if check_ulp:
            # against the oracle rounded to bf16: at most one bf16 step apart, plus the fp32 rounding of
            # the O(w) terms the gradient is a difference of (w = 1, or 1/n_valid for the mean)
            scale = 1.0 if reduction == cb.REDUCE_SUM else 1.0 / max(int(ref.counters[0]), 1)
            step = bf16_ulp(np.maximum(np.abs(ref.grad), np.abs(g)))
            assert np.all(np.abs(g - bf16_round(ref.grad)) <= step * 1.0001 + 1e-6 * scale)
    return plan, out, ref
