"""GPU parity at the full sizes of the two large workloads, in the launch configuration bench.py
times (MSE distance, mean over valid rows, counters on).  The oracle computes every per-row loss,
the reduced loss and the counters for the whole batch, and the gradient for three row ranges
(first, middle, last rows, which include padded rows)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2010_02838_b200 import binding as cb
from paper_2010_02838_b200 import synth

from helpers import bf16_ulp, to_device

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("idx", [4, 5])
def test_full_size_workload(idx):
    w = synth.WORKLOADS[idx]
    free, _ = torch.cuda.mem_get_info()
    if free < 1.3 * w.algorithmic_bytes():
        pytest.skip("not enough free device memory for the full workload")
    own, peers, labels, mask = synth.make_inputs(w)
    d_own, d_peers = to_device(own), [to_device(p) for p in peers]
    plan = cb.Plan(d_own, d_peers, to_device(labels), to_device(mask), alpha=w.alpha, temperature=w.temperature,
                   label_smoothing=w.label_smoothing)
    assert plan.regime == {4: "tma", 5: "stream"}[idx]      # the launch configuration the benchmark times
    out = plan.run()
    torch.cuda.synchronize()
    assert out.status.item() == 0
    kw = dict(alpha=w.alpha, temperature=w.temperature, label_smoothing=w.label_smoothing)
    ref = oracle.codistill(own, peers, labels, mask, want_grad=False, **kw)
    assert out.counters.cpu().tolist() == ref.counters.tolist()                  # integers: bit-exact
    assert abs(out.loss.item() - ref.loss) <= 2e-3 * abs(ref.loss)
    np.testing.assert_allclose(out.row_loss.cpu().numpy(), ref.row_loss, rtol=2e-3, atol=2e-7)
    n_valid = int(ref.counters[0])
    R = w.rows
    for lo in (0, R // 2 - 16, R - 32):
        part = oracle.codistill(own, peers, labels, mask, grad_rows=(lo, lo + 32), **kw)
        g = out.grad[lo:lo + 32].double().cpu().numpy()
        # under the mean every element is scaled by 1/n_valid: compare at that scale (values whose
        # scaled magnitude exceeds 1 are bounded by bf16 rounding itself, as in helpers.compare)
        err = np.abs(g - part.grad) * n_valid
        assert np.all(err <= np.maximum(2e-3, 0.75 * bf16_ulp(part.grad * n_valid)))
        dead = np.flatnonzero(mask[lo:lo + 32] == 0)
        assert np.all(g[dead] == 0)
    del plan, out, d_own, d_peers
    torch.cuda.empty_cache()
