"""Prediction compression and exchange (Section 3): the bfloat16 packing against its definition, the
effect of the packing on the distillation distance, the device kernels against the restatement (GPU),
and the exchange schedule with two gloo ranks on the CPU."""
import os
import socket
import sys

import numpy as np
import pytest
import torch

import oracle
from oracle import predictions as ref

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


# ---------------------------------------------------------------- the restatement against hand values
def test_packing_rounds_to_nearest_even_on_hand_values():
    one = 0x3F80                                      # 1.0 in bf16
    assert ref.pack_one(1.0) == one
    assert ref.pack_one(1.0 + 2.0 ** -8) == one       # exactly half-way between 1 and 1 + 2^-7: tie goes to the even pattern
    assert ref.pack_one(1.0 + 2.0 ** -8 + 2.0 ** -20) == one + 1
    assert ref.pack_one(1.0 + 3 * 2.0 ** -8) == one + 2   # half-way between odd 0x3F81 and even 0x3F82: up to even
    assert ref.pack_one(-1.0 - 2.0 ** -8) == 0xBF80
    assert ref.pack_one(0.0) == 0 and ref.pack_one(-0.0) == 0x8000
    assert ref.pack_one(float("inf")) == 0x7F80 and ref.pack_one(float("-inf")) == 0xFF80
    assert ref.pack_one(3.3895313892515355e38) == 0x7F7F      # the largest bf16 stays finite
    assert ref.pack_one(3.4e38) == 0x7F80                      # beyond the last half-way point: infinity
    b = ref.pack_one(float("nan"))
    assert (b & 0x7F80) == 0x7F80 and (b & 0x007F) != 0        # still a NaN
    assert ref.unpack_one(0x3F81) == 1.0 + 2.0 ** -7


def test_vectorised_packing_is_the_elementwise_definition():
    g = np.random.default_rng(3)
    x = np.concatenate([g.standard_normal(4000).astype(np.float32) * 3, np.float32([0, -0.0, 1 + 2 ** -8, 1e-40, -1e-39, 65504.0]),
                        (1 + np.arange(64) * 2.0 ** -9).astype(np.float32)])
    assert ref.pack(x).tolist() == [ref.pack_one(float(v)) for v in x]
    back = ref.unpack(ref.pack(x))
    assert np.all(np.abs(back.astype(np.float64) - x) <= 2.0 ** -8 * np.abs(x) + 2.0 ** -134)   # half a bf16 step (8 significant bits)
    assert np.array_equal(ref.pack(back), ref.pack(x))                                            # idempotent


def test_effect_of_packing_on_the_distance_is_within_its_bound():
    """MSE distance against packed peers: |D' - D| <= 1/C sum_c (2 |z_c - v_c| e_c + e_c^2), e_c = 2^-8 |v_c|
    (half a step of an 8-bit significand)."""
    g = np.random.default_rng(8)
    rows, C = 6, 1000
    own = (2 * g.standard_normal((rows, C))).astype(np.float32)
    peer = (own + 0.5 * g.standard_normal((rows, C))).astype(np.float32)
    packed = ref.unpack(ref.pack(peer)).reshape(rows, C)
    labels = g.integers(0, C, rows).astype(np.int32)
    kw = dict(alpha=1.0, reduction=oracle.REDUCE_SUM, want_grad=False)
    d_exact = oracle.codistill(own, [peer], labels, **kw).row_loss - oracle.codistill(own, [], labels, **kw).row_loss
    d_packed = oracle.codistill(own, [packed], labels, **kw).row_loss - oracle.codistill(own, [], labels, **kw).row_loss
    e = 2.0 ** -8 * np.abs(peer.astype(np.float64))
    bound = (2 * np.abs(own.astype(np.float64) - peer) * e + e * e).mean(1)
    assert np.all(np.abs(d_packed - d_exact) <= bound)
    assert np.all(np.abs(d_packed - d_exact) > 0)       # and the packing does change the distance


# ---------------------------------------------------------------- device kernels
@pytest.mark.gpu
@pytest.mark.parametrize("rows,C,pitch", [(7, 1000, 1000), (5, 1003, 1003), (3, 10, 16), (64, 32768, 32768), (1, 1, 1), (0, 8, 8)])
def test_device_packing_matches_the_definition(rows, C, pitch):
    from paper_2010_02838_b200 import binding as cb
    g = np.random.default_rng(rows * 31 + C)
    x = (3 * g.standard_normal((rows, pitch))).astype(np.float32)
    if rows:
        x[0, : min(C, 4)] = np.float32([1 + 2 ** -8, 1 + 3 * 2 ** -8, -1 - 2 ** -8, 0.0][: min(C, 4)])
    d = torch.from_numpy(x).cuda()
    out = torch.full((rows, pitch), 7.0, dtype=torch.bfloat16, device="cuda")
    cb.pack_predictions(d[:, :C], out[:, :C])
    torch.cuda.synchronize()
    got = out.view(torch.int16).cpu().numpy().view(np.uint16)
    assert np.array_equal(got[:, :C], ref.pack(x[:, :C]).reshape(rows, C))
    assert np.all(got[:, C:] == 0x40E0)                                   # the pitch padding (7.0) is untouched
    wide = torch.full((rows, pitch), -3.0, dtype=torch.float32, device="cuda")
    cb.unpack_predictions(out[:, :C], wide[:, :C])
    torch.cuda.synchronize()
    assert np.array_equal(wide.cpu().numpy()[:, :C], ref.unpack(ref.pack(x[:, :C])).reshape(rows, C))
    assert torch.all(wide[:, C:] == -3.0)


# ---------------------------------------------------------------- the exchange schedule on two CPU ranks
def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    from paper_2010_02838_b200 import exchange
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    rows, C, period = 12, 40, 3
    labels = np.random.default_rng(99).integers(0, C, rows).astype(np.int32)       # coordinated sampling: same minibatch
    ex = exchange.PredictionExchange(period=period)
    log = []
    for step in range(7):
        own = np.random.default_rng(1000 * step + rank).standard_normal((rows, C)).astype(np.float32)
        peers = ex.peers_for_step(torch.from_numpy(own))
        other = np.random.default_rng(1000 * step + (1 - rank)).standard_normal((rows, C)).astype(np.float32)
        if step % period == 0:
            assert len(peers) == world - 1 and np.array_equal(peers[0].numpy(), other)      # the other rank's bits
        else:
            assert peers == []
        res = oracle.codistill(own, [p.numpy() for p in peers], labels, alpha=1.0, reduction=oracle.REDUCE_SUM)
        plain = oracle.codistill(own, [], labels, alpha=1.0, reduction=oracle.REDUCE_SUM)
        log.append((len(peers), res.loss, plain.loss))
    bits = ex.bits_sent_per_step(classes=1000, batch_per_device=32)
    q.put((rank, log, bits))
    dist.barrier()
    dist.destroy_process_group()


def test_periodic_exchange_between_two_model_groups():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, log, bits in got:
        assert [n for n, _, _ in log] == [1, 0, 0, 1, 0, 0, 1]
        for n_peers, loss, plain in log:
            if n_peers == 0:
                assert loss == plain                       # the term is left out on the steps in between
            else:
                assert loss > plain                        # the distance between different models is positive
        assert bits == pytest.approx(1.024e6 / 3)          # (n-1) b_pred B / T with b_pred = 3.2e4, B = 32, T = 3
