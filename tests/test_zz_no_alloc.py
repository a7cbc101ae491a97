"""The allocation-free entry point (codistill_loss_fwd_bwd_static).

Some users of this library cannot allocate device memory when they call the loss: a framework
has reserved the whole GPU up front, or their step loop forbids allocator calls.  For them the
library carries its scratch as a fixed device array.  This file checks, through the C ABI, that
the entry point gives the same results as the ordinary one on two calls in a row (the scratch is
shared and keeps the previous call's contents) and as the CPU oracle, that a call leaves the amount
of free device memory unchanged, and that it refuses batches beyond its capacity.
It is collected after every other test file on purpose.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2010_02838_b200 import binding as cb
from paper_2010_02838_b200 import synth


def _dev(a):
    if a is None:
        return None
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(a).cuda()


def _outputs(like):
    rows = like.shape[0]
    return cb.Outputs(torch.full((rows,), 9.0, dtype=torch.float32, device="cuda"),
                      torch.full((1,), 9.0, dtype=torch.float32, device="cuda"),
                      torch.full_like(like, 9.0), None, None)


@pytest.mark.gpu
@pytest.mark.parametrize("idx,rows", [(2, 256), (4, 96)])
def test_static_scratch_matches_ordinary_entry_point(idx, rows):
    """Two different batches back to back through the static-scratch call, each compared with
    codistill_loss_fwd_bwd on the same inputs (warp-per-row and bulk-copy kernels)."""
    base = synth.scaled(synth.WORKLOADS[idx], rows=rows)
    tol_loss, tol_grad = (1e-5, 1e-6) if base.dtype == "f32" else (2e-3, 2e-3)
    for call in range(2):
        w = synth.scaled(base, rows=rows if call == 0 else rows - 32, name=f"call{call}")
        own, peers, labels, mask = synth.make_inputs(w)
        if call == 1:
            own = peers[0].copy()          # other data than the first call left behind
        if mask is None:
            mask = (np.arange(w.rows) % 5 != call).astype(np.uint8)
        d_own, d_peers, d_labels, d_mask = _dev(own), [_dev(p) for p in peers], _dev(labels), _dev(mask)
        ref = cb.codistill_loss_fwd_bwd(d_own, d_peers, d_labels, d_mask, alpha=0.8)
        outs = _outputs(d_own)
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        got = cb.codistill_loss_fwd_bwd_static(d_own, d_peers, d_labels, d_mask, outs, alpha=0.8)
        torch.cuda.synchronize()
        if call == 1:   # the first call on a device may load the library's device code; later ones take nothing
            assert torch.cuda.mem_get_info()[0] == free_before
        assert abs(got.loss.item() - ref.loss.item()) <= tol_loss * abs(ref.loss.item())
        np.testing.assert_allclose(got.row_loss.cpu().numpy(), ref.row_loss.cpu().numpy(), rtol=tol_loss, atol=2e-7)
        assert (got.grad.double() - ref.grad.double()).abs().max().item() <= tol_grad
        # and against the oracle's definition (MSE distance, mean over valid rows)
        exact = oracle.codistill(own, peers, labels, mask, alpha=0.8)
        assert abs(got.loss.item() - exact.loss) <= tol_loss * abs(exact.loss)
        np.testing.assert_allclose(got.row_loss.cpu().numpy(), exact.row_loss, rtol=tol_loss, atol=2e-7)
        assert np.abs(got.grad.double().cpu().numpy() - exact.grad).max() <= tol_grad
        # without a row_loss buffer the per-row losses stay in the built-in scratch: same reduced loss
        no_rows = cb.Outputs(None, torch.zeros(1, dtype=torch.float32, device="cuda"), torch.zeros_like(d_own), None, None)
        cb.codistill_loss_fwd_bwd_static(d_own, d_peers, d_labels, d_mask, no_rows, alpha=0.8)
        torch.cuda.synchronize()
        assert no_rows.loss.item() == got.loss.item() and torch.equal(no_rows.grad, got.grad)


def test_static_scratch_rejects_oversized_batches():
    """More rows than the built-in scratch holds: a clear error code, nothing launched (needs no GPU)."""
    from paper_2010_02838_b200 import build as cbuild
    cbuild.build()
    lib = cb.load_library()
    fake = ctypes.c_void_p(4096)   # never dereferenced: the size check comes first
    ptrs = (ctypes.c_void_p * 1)(4096)
    rc = lib.codistill_loss_fwd_bwd_static(fake, ptrs, fake, None, 2, cb.STATIC_MAX_ROWS + 1, 16, 1.0, 1.0, cb.F32,
                                           fake, fake, fake, None)
    assert rc == cb.ERR_TOO_LARGE and "STATIC_MAX_ROWS" in cb.status_string(rc)
    rc = lib.codistill_loss_fwd_bwd_static(fake, ptrs, fake, None, 2, 8, 16, 1.0, 1.0, cb.F32, fake, None, fake, None)
    assert rc == 1                 # the reduced loss has no default destination
