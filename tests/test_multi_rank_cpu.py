"""The N > 1 path of the benchmark shards nothing on the data path: every rank owns a whole batch.
Its host logic (rank-distinct seeds, max-over-ranks of the device time, whole-job throughput) is
exercised here with two gloo ranks on the CPU; no GPU is needed."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import dataclasses
    import oracle
    from paper_2010_02838_b200 import synth
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = dataclasses.replace(synth.scaled(synth.WORKLOADS[4], rows=64, classes=512), seed=rank)  # rank-distinct batch
    own, peers, labels, mask = synth.make_inputs(w)
    res = oracle.codistill(own, peers, labels, mask, alpha=w.alpha, label_smoothing=w.label_smoothing)
    ms = torch.tensor([1.0 + rank], dtype=torch.float64)          # pretend device time of this rank
    dist.all_reduce(ms, op=dist.ReduceOp.MAX)
    rows_per_s = world * w.rows / (ms.item() * 1e-3)
    q.put((rank, float(res.loss), int(own[0, 0]), ms.item(), rows_per_s))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_independent_batches_and_max_time():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, loss0, first0, ms0, v0), (r1, loss1, first1, ms1, v1) = got
    assert (r0, r1) == (0, 1)
    assert first0 != first1 and loss0 != loss1            # different seeds: different batches
    assert ms0 == ms1 == 2.0                              # max over ranks
    assert v0 == v1 == 2 * 64 / 2e-3                      # whole-job rows/s


def test_bench_starts_one_rank_per_gpu_when_asked_outside_a_launcher():
    """`bench.py --gpus N` run as a plain script re-launches itself under torchrun with N local ranks."""
    sys.path.insert(0, ROOT)
    import bench
    cmd = bench.torchrun_command(["--gpus", "4", "--steps", "7"], 4, port=29431)
    assert cmd[:3] == [sys.executable, "-m", "torch.distributed.run"]
    assert "--nproc-per-node=4" in cmd and "--nnodes=1" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[cmd.index("--master-port") + 1] == "29431"
    assert cmd[-5:] == [os.path.join(ROOT, "bench.py"), "--gpus", "4", "--steps", "7"]
