"""GPU parity of the two long-row kernels, each forced through CODISTILL_REGIME on shapes both serve
(the default choice depends on the row length): the direct-load "stream" kernel and the staged "tma"
kernel; and of the default choice on rows too long for shared memory."""
import numpy as np
import pytest
import torch

from paper_2010_02838_b200 import binding as cb
from paper_2010_02838_b200 import synth

from helpers import compare

pytestmark = pytest.mark.gpu


def rand_inputs(seed, rows, C, n, dtype, scale=1.5):
    g = np.random.default_rng(seed)
    mk = lambda: (scale * g.standard_normal((rows, C))).astype(np.float32)
    own, peers = mk(), [mk() for _ in range(n - 1)]
    labels = g.integers(0, C, rows).astype(np.int32)
    if dtype == "bf16":
        own, peers = synth.f32_to_bf16_bits(own), [synth.f32_to_bf16_bits(p) for p in peers]
    return own, peers, labels


@pytest.fixture(params=["stream", "tma"])
def forced_regime(request, monkeypatch):
    monkeypatch.setenv("CODISTILL_REGIME", request.param)
    return request.param


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("C,n", [(32768, 2), (50257, 8), (4099, 3), (8192, 1), (20011, 4), (33000, 3)])
@pytest.mark.parametrize("reduction", [0, 1])
def test_forced_regime_parity(forced_regime, dtype, C, n, reduction):
    if dtype == "bf16" and C * 2 < 8192:
        pytest.skip("row shorter than the long-row kernels take")
    rows = 21
    # a 201 KB fp32 row does not fit the staged kernel's shared-memory buffer: the request falls through
    expect = "stream" if (dtype == "f32" and C * 4 > 180000) else forced_regime
    own, peers, labels = rand_inputs(C + n, rows, C, n, dtype)
    mask = (np.arange(rows) % 6 != 2).astype(np.uint8)
    # labels on the first and last columns exercise the ragged segments of unaligned rows
    labels[0], labels[1] = 0, C - 1
    compare(own, peers, labels, mask, alpha=0.7, label_smoothing=0.1 if n == 2 else 0.0,
            peer_reduce=cb.PEERS_MEAN_TARGET if n == 4 else cb.PEERS_PAIRWISE_MEAN,
            reduction=reduction, expect_regime=expect)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_forced_regime_ties_and_edges(forced_regime, dtype):
    """Planted maxima: ties inside a segment, across segments, on the first and last column of an
    unaligned row, and -0.0 against +0.0; the counters must match the oracle bit for bit."""
    rows, C, n = 16, 9001 if dtype == "f32" else 9003, 3
    own, peers, labels = rand_inputs(5, rows, C, n, dtype, scale=1.0)

    def plant(a, r, cols, val):
        v = np.float32(val)
        for c in cols:
            if a.dtype == np.uint16:
                a[r, c] = synth.f32_to_bf16_bits(np.array([v], dtype=np.float32))[0]
            else:
                a[r, c] = v
    for r in range(rows):
        cols = [(r * 577) % C, (r * 577 + 3) % C, C - 1 - (r % 3), r % 2]
        plant(own, r, cols, 9.0)
        plant(peers[0], r, cols[1:], 9.0)          # peer 0 ties on a later column: agrees only if its first max is the own arg-max
        plant(peers[1], r, [min(cols)], 9.0)       # peer 1 peaks on the own arg-max
    own_z = own.copy()
    compare(own, peers, labels, None, alpha=1.0, reduction=cb.REDUCE_SUM, expect_regime=forced_regime)
    assert np.array_equal(own, own_z)


def test_very_long_rows_take_the_stream_kernel():
    """A vocabulary too long for the shared-memory row buffer: served by the direct-load kernel by default."""
    rows, C, n = 6, 150001, 2
    own, peers, labels = rand_inputs(11, rows, C, n, "bf16")
    mask = np.array([1, 1, 0, 1, 1, 1], dtype=np.uint8)
    plan, out, ref = compare(own, peers, labels, mask, alpha=1.0, label_smoothing=0.05, reduction=cb.REDUCE_SUM,
                             expect_regime="stream")
    # guard band: nothing is written outside the gradient rows (the base stays 16-byte aligned)
    g = torch.full((rows * C + 64,), 3.0, dtype=torch.bfloat16, device="cuda")
    plan.params.grad_logits = g[32:].data_ptr()
    plan.run()
    torch.cuda.synchronize()
    assert plan.regime == "stream"
    assert torch.all(g[:32].float() == 3.0) and torch.all(g[32 + rows * C:].float() == 3.0)
    assert torch.equal(g[32:32 + rows * C].view(rows, C), out.grad)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("peer_reduce", [cb.PEERS_PAIRWISE_MEAN, cb.PEERS_MEAN_TARGET])
@pytest.mark.parametrize("C,n,temperature", [(32768, 2, 1.0), (50257, 4, 2.0), (9001, 8, 0.7), (8192, 1, 3.0)])
def test_kl_form_on_long_rows(dtype, peer_reduce, C, n, temperature):
    """The softmax-KL distance on long rows is served by the direct-load kernel (one more pass for the
    peers' softmax statistics)."""
    rows = 13
    own, peers, labels = rand_inputs(3 * C + n, rows, C, n, dtype)
    mask = (np.arange(rows) % 5 != 3).astype(np.uint8)
    labels[0], labels[1] = 0, C - 1
    for reduction in (cb.REDUCE_SUM, cb.REDUCE_MEAN_VALID):
        compare(own, peers, labels, mask, alpha=0.9, temperature=temperature, label_smoothing=0.05,
                dist=cb.DIST_KL_SOFTMAX, peer_reduce=peer_reduce, reduction=reduction, expect_regime="stream")


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("peer_reduce", [cb.PEERS_PAIRWISE_MEAN, cb.PEERS_MEAN_TARGET])
@pytest.mark.parametrize("C,n", [(32768, 2), (50257, 4), (9001, 8), (8192, 1)])
def test_centred_mse_on_long_rows(dtype, peer_reduce, C, n):
    """The centred MSE distance on long rows is served by the direct-load kernel (one more pass for the
    peers' class sums)."""
    rows = 13
    own, peers, labels = rand_inputs(5 * C + n, rows, C, n, dtype)
    peers = [p if p.dtype == np.uint16 else (p + np.float32(0.5 * (j + 1))) for j, p in enumerate(peers)]  # shifted peers
    mask = (np.arange(rows) % 5 != 3).astype(np.uint8)
    labels[0], labels[1] = 0, C - 1
    for reduction in (cb.REDUCE_SUM, cb.REDUCE_MEAN_VALID):
        compare(own, peers, labels, mask, alpha=0.9, label_smoothing=0.05, dist=cb.DIST_MSE_CENTRED,
                peer_reduce=peer_reduce, reduction=reduction, expect_regime="stream")
