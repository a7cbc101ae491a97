#!/usr/bin/env python
"""Benchmark of the fused codistillation loss forward + gradient (one JSON line on stdout).

A step is one pass of the whole hot path (row statistics, task loss, distillation distance,
gradient, per-row and reduced loss, counters) over one batch of synthetic logits.  The default
workload is the translation-head shape the headline metric is quoted on: n = 2 models,
8192 token rows x 32768 classes, bf16, 10 % padded rows, label smoothing 0.1.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 1..5] [--impl ours|reference]

N > 1 runs under torchrun, one process per GPU; every rank processes its own batch of the same
shape (weak scaling, no collective on the data path; NCCL is used for the barrier and the
max-over-ranks of the device time only).
"""
from __future__ import annotations

import argparse
import ctypes
import hashlib
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "codistill_loss_fwd_bwd_rows_per_s"
UNIT = "rows/s"
FALLBACK_HBM_GBS = 6650.0


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", type=int, default=4, choices=[1, 2, 3, 4, 5])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--dist", default="mse", choices=["mse", "kl", "mse_centred"])
    ap.add_argument("--rows", type=int, default=0, help="run a smaller batch of the same recipe (profiling aid)")
    ap.add_argument("--all-models", action="store_true",
                    help="one call computes the objectives of all n models (codistill_loss_fwd_bwd_all); rows/s then counts "
                         "model-rows (n x rows per step)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sustain", type=float, default=3.0,
                    help="seconds of back-to-back steps timed in chunks with the SM clock read after each (0: skip)")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the legs beside the headline (sustained run, graph replay, basic entry point)")
    return ap.parse_args()


def workload_config(idx, w, dist):
    return {"workload": f"config{idx}:{w.name}",
            "n": w.n, "rows": w.rows, "classes": w.classes, "alpha": w.alpha, "temperature": w.temperature,
            "label_smoothing": w.label_smoothing, "padded_rows": w.n_padded, "dist": dist,
            "reduction": "mean_valid", "l2": "inputs larger than L2 (no flush needed)" if
            w.algorithmic_bytes() > 3 * 126e6 else "L2-resident: latency-bound, roofline fraction not meaningful"}


# ------------------------------------------------------------------ clocks
class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "100", "-i", str(self.index)],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx = float(f[1])
            except ValueError:
                continue
            for name, val in zip(["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"], f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


# ------------------------------------------------------------------ peaks and stored traffic
def hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback (earlier pool measurement)"


def kernel_source_hash(files):
    """Hash of the named kernel sources (the files a stored ncu capture depends on)."""
    h = hashlib.sha256()
    d = os.path.join(ROOT, "paper_2010_02838_b200", "csrc")
    for f in sorted(files):
        h.update(open(os.path.join(d, f), "rb").read())
    return h.hexdigest()[:16]


def stored_traffic(workload_idx, dist, all_models, w):
    """DRAM bytes per launch of the dominant kernel from the committed ncu record (profiles/dram_traffic.json),
    or None when there is no record or the kernel sources changed since the capture.  A record holds the
    counters of the second of two consecutive launches (caches left alone between them) on a reduced batch of
    the same recipe; reads are scaled by valid rows, writes by rows."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    if not os.path.exists(path):
        return None
    try:
        rec = json.load(open(path)).get(f"config{workload_idx}_{dist}" + ("_all" if all_models else ""))
        if not rec or rec.get("source_hash") != kernel_source_hash(rec["sources"]):
            return None
        cap = rec["capture"]
        reads = cap["dram_bytes_read"] * (w.rows - w.n_padded) / cap["valid_rows"]
        writes = cap["dram_bytes_write"] * w.rows / cap["rows"]
        return int(reads + writes)
    except Exception:
        return None


# ------------------------------------------------------------------ reference arm: the CPU oracle
def oracle_sample_rows(w):
    """Rows per timed oracle call: about 4e8 logit elements (several core-seconds of CPU work per call)."""
    per_row = w.classes * w.n
    rows = max(1, min(w.rows, int(4.0e8 // per_row)))
    if w.tokens_per_seq:
        rows = max(w.tokens_per_seq, rows // w.tokens_per_seq * w.tokens_per_seq)
    return min(rows, w.rows)


def time_oracle(w, dist, steps, warmup, min_seconds=0.0):
    """Times the oracle as it stands on a bounded sample; with min_seconds the call is repeated until
    that much wall time has been spent (at least `steps` calls)."""
    import oracle
    from paper_2010_02838_b200 import synth
    rows = oracle_sample_rows(w)
    own, peers, labels, mask = synth.make_inputs(w, 0, rows)
    kw = dict(alpha=w.alpha, temperature=w.temperature, label_smoothing=w.label_smoothing,
              dist={"mse": oracle.DIST_MSE, "kl": oracle.DIST_KL, "mse_centred": oracle.DIST_MSE_CENTRED}[dist])
    for _ in range(warmup):
        oracle.codistill(own, peers, labels, mask, **kw)
    t0 = time.perf_counter()
    done = 0
    while done < steps or (time.perf_counter() - t0) < min_seconds:
        oracle.codistill(own, peers, labels, mask, **kw)
        done += 1
    dt = (time.perf_counter() - t0) / max(done, 1)
    return rows / dt, dt, rows, oracle.max_threads(), done


def run_reference(args):
    from paper_2010_02838_b200 import synth
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = synth.WORKLOADS[args.workload]
    if args.rows:
        w = synth.scaled(w, rows=args.rows)
    steps, warmup = max(1, args.steps), max(0, args.warmup)
    value, dt, rows, cores, _ = time_oracle(w, args.dist, steps, warmup)
    sample = f"first {rows} rows of the workload per step, all {w.n} models, fp64 oracle as it stands"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic", "config": workload_config(args.workload, w, args.dist),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------ our arm
def to_device(a, torch):
    import numpy as np
    if a is None:
        return None
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(a).cuda()


def make_device_inputs(w, torch, seed_offset=0):
    """Generate the workload slice by slice on the host and upload it (bounded host memory)."""
    import dataclasses
    import numpy as np
    from paper_2010_02838_b200 import synth
    w = dataclasses.replace(w, seed=w.seed + seed_offset)
    tdt = torch.float32 if w.dtype == "f32" else torch.bfloat16
    models = [torch.empty((w.rows, w.classes), dtype=tdt, device="cuda") for _ in range(w.n)]
    step = max(1, int(2.0e8 // w.classes))
    for r0 in range(0, w.rows, step):
        r1 = min(w.rows, r0 + step)
        for k in range(w.n):
            models[k][r0:r1].copy_(to_device(synth.make_model_logits(w, k, r0, r1), torch))
    labels = to_device(synth.make_labels(w), torch)
    mask = to_device(synth.make_mask(w), torch)
    return w, models, labels, mask


def run_ours(args):
    import numpy as np
    import torch
    import torch.distributed as dist_pkg
    from paper_2010_02838_b200 import binding as cb
    from paper_2010_02838_b200 import build as cbuild
    from paper_2010_02838_b200 import synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the codistillation kernels have no CPU path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist_pkg.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if rank == 0:
        cbuild.build()
    if world > 1:
        dist_pkg.barrier()
    cb.load_library()

    w0 = synth.WORKLOADS[args.workload]
    if args.rows:
        w0 = synth.scaled(w0, rows=args.rows)
    dist_code = {"mse": cb.DIST_MSE_LOGITS, "kl": cb.DIST_KL_SOFTMAX, "mse_centred": cb.DIST_MSE_CENTRED}[args.dist]
    w, models, labels, mask = make_device_inputs(w0, torch, seed_offset=rank)   # each rank: its own batch
    if args.all_models:
        plan = cb.AllPlan(models, labels, mask, alpha=w.alpha, temperature=w.temperature,
                          label_smoothing=w.label_smoothing, dist=dist_code)
        plan.regime = "all-models"
    else:
        plan = cb.Plan(models[0], models[1:], labels, mask, alpha=w.alpha, temperature=w.temperature,
                       label_smoothing=w.label_smoothing, dist=dist_code)
    stream = torch.cuda.current_stream()

    def barrier():
        if world > 1:
            dist_pkg.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        plan.run(stream)
    barrier()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record(stream)
    for _ in range(args.steps):
        plan.run(stream)
    ev1.record(stream)
    barrier()
    ms_total = ev0.elapsed_time(ev1)
    clocks = sampler.stop() if rank == 0 else None
    if world > 1:
        t = torch.tensor([ms_total], device="cuda", dtype=torch.float64)
        dist_pkg.all_reduce(t, op=dist_pkg.ReduceOp.MAX)
        ms_total = float(t.item())
    ms_step = ms_total / args.steps
    rows_per_step = w.rows * (w.n if args.all_models else 1)
    rows_per_s = world * rows_per_step / (ms_step * 1e-3)
    status = int(plan.out.status.item())
    if status != 0:
        raise RuntimeError(f"device status {status} after the timed region")

    extras = {}
    if rank == 0 and world == 1 and not args.no_extras:
        extras = run_extras(args, w, plan, models, labels, mask, cb, torch, stream, ms_step, local_rank)

    # ---- end to end through the host-buffer entry point (pinned host memory, copies inside the timed region)
    e2e = None
    if not args.no_e2e and not args.all_models:
        e2e = run_e2e(args, w, models, labels, mask, cb, torch, world, barrier, dist_code)

    if rank != 0:
        if world > 1:
            dist_pkg.destroy_process_group()
        return

    peak, peak_src = hbm_peak()
    alg_bytes = w.algorithmic_bytes(skip_masked_reads=True)
    launches_per_step = 2   # prep kernel + main kernel (the main kernel's last CTA does the final reduction)
    note = ("algorithmic bytes with masked-row reads skipped: n*R_valid*C*s + R*C*s + 9R; "
            "duration = step time (prep + main kernel) from CUDA events on the launch stream")
    if args.all_models:
        es = 4 if w.dtype == "f32" else 2
        r_valid = w.rows - w.n_padded
        alg_bytes = w.n * (r_valid + w.rows) * w.classes * es + 9 * w.rows * w.n
        launches_per_step = 3   # prep kernel + all-models kernel + final reduction of the n models
        note = ("all n objectives per step; algorithmic bytes = every tensor read once and every gradient written "
                "once: n*(R_valid + R)*C*s (the kernel reads each tensor twice: 3n passes; n single calls move n*(n+1))")
    achieved = alg_bytes / (ms_step * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": rows_per_s, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": dict(workload_config(args.workload, w0, args.dist), **({"all_models": True} if args.all_models else {})),
        "io_dtype": w.dtype, "kernel_regime": plan.regime,
        "hbm_gbs_algorithmic": achieved,
        "hbm_gbs_dense_formula": None if args.all_models else w.algorithmic_bytes() / (ms_step * 1e-3) / 1e9,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": stored_traffic(args.workload, args.dist, args.all_models, w), "peak_source": peak_src,
                     "bytes_per_launch": alg_bytes,
                     "note": note},
        "frac_of_nominal_8TBs": achieved / 8000.0,
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
    }
    if clocks and clocks.get("sm_mhz"):
        line["ms_x_sm_mhz"] = ms_step * clocks["sm_mhz"]     # for an issue-bound kernel: SM cycles per step / 1000
    line.update(extras)
    if not args.no_cpu_baseline:
        v, dt, rows, cores, calls = time_oracle(w0, args.dist, 2, 1, min_seconds=12.0)
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": f"first {rows} rows of the workload, all {w.n} models, {calls} calls of {dt:.2f} s "
                                          f"({calls * dt * cores:.0f} core-seconds)"}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist_pkg.destroy_process_group()


def sm_clock_reader(index):
    """Returns a function that reads the current SM clock in MHz through NVML (reading only), or None."""
    try:
        import pynvml
        pynvml.nvmlInit()
        handle = pynvml.nvmlDeviceGetHandleByIndex(index)
        return lambda: int(pynvml.nvmlDeviceGetClockInfo(handle, pynvml.NVML_CLOCK_SM))
    except Exception:
        return None


def run_extras(args, w, plan, models, labels, mask, cb, torch, stream, ms_step, device_index):
    """Legs beside the headline, each timed with CUDA events on the launch stream:
    - sustained: back-to-back steps for args.sustain seconds in chunks of about 50 ms, the SM clock read
      after each chunk; time per step by clock bin, so that the dependence on the clock is on record;
    - graph_replay (workloads that fit the L2, where launch latency dominates): the same call captured in a
      CUDA graph, 20 steps per graph;
    - basic_entry_point: the plain codistill_loss_fwd_bwd call (scratch from the stream-ordered allocator,
      no counters) on the same tensors, single-model workloads with dense MSE only."""
    out = {}
    ev = lambda: torch.cuda.Event(enable_timing=True)
    if args.sustain > 0:
        read_clock = sm_clock_reader(device_index)
        chunk = max(1, int(50.0 / max(ms_step, 1e-3)))
        bins, t_all, t0 = {}, [], time.perf_counter()
        while time.perf_counter() - t0 < args.sustain:
            e0, e1 = ev(), ev()
            e0.record(stream)
            for _ in range(chunk):
                plan.run(stream)
            e1.record(stream)
            e1.synchronize()
            mhz = read_clock() if read_clock else None
            ms = e0.elapsed_time(e1) / chunk
            t_all.append(ms)
            bins.setdefault(mhz, []).append(ms)
        t_all.sort()
        out["sustained"] = {
            "seconds": round(time.perf_counter() - t0, 2), "steps": chunk * len(t_all),
            "ms_per_step_median": t_all[len(t_all) // 2], "ms_per_step_max": t_all[-1],
            "by_sm_mhz": {str(k): {"chunks": len(v), "ms_per_step_median": sorted(v)[len(v) // 2]}
                          for k, v in sorted(bins.items(), key=lambda kv: -(kv[0] or 0))},
            "note": "chunks of about 50 ms of back-to-back steps; SM clock read through NVML after each chunk"}
    if w.algorithmic_bytes() <= 3 * 126e6:
        try:
            per_graph = 20
            side = torch.cuda.Stream()
            side.wait_stream(stream)
            with torch.cuda.stream(side):
                plan.run(side)
            stream.wait_stream(side)
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                for _ in range(per_graph):
                    plan.run(torch.cuda.current_stream())
            for _ in range(3):
                g.replay()
            reps = max(5, args.steps // per_graph)
            e0, e1 = ev(), ev()
            e0.record()
            for _ in range(reps):
                g.replay()
            e1.record()
            e1.synchronize()
            out["graph_replay"] = {"ms_per_step": e0.elapsed_time(e1) / (reps * per_graph), "steps_per_graph": per_graph,
                                   "replays": reps, "note": "the same C-ABI call captured in a CUDA graph"}
        except Exception as exc:   # capture is a convenience of this benchmark, not of the library's contract
            out["graph_replay"] = {"error": str(exc)[:200]}
    if not args.all_models and args.dist == "mse":
        outs = cb.Outputs(torch.empty(w.rows, dtype=torch.float32, device="cuda"),
                          torch.empty(1, dtype=torch.float32, device="cuda"), torch.empty_like(models[0]), None, None)
        call = lambda: cb.codistill_loss_fwd_bwd(models[0], models[1:], labels, mask, alpha=w.alpha,
                                                 temperature=w.temperature, out=outs, stream=stream)
        for _ in range(3):
            call()
        e0, e1 = ev(), ev()
        e0.record(stream)
        for _ in range(args.steps):
            call()
        e1.record(stream)
        e1.synchronize()
        out["basic_entry_point"] = {"ms_per_step": e0.elapsed_time(e1) / args.steps, "api": "codistill_loss_fwd_bwd",
                                    "note": "same tensors; this call has no label smoothing and no counters, and takes "
                                            "its scratch from the stream-ordered allocator"}
    return out


def run_e2e(args, w, models, labels, mask, cb, torch, world, barrier, dist_code):
    """Same metric through codistill_loss_fwd_bwd_host: inputs start in pinned host memory, every
    output (gradient, per-row and reduced loss, counters) ends in pinned host memory."""
    n, rows, C = w.n, w.rows, w.classes
    h_models = [m.cpu().pin_memory() for m in models]
    h_labels, h_mask = labels.cpu().pin_memory(), (mask.cpu().pin_memory() if mask is not None else None)
    h_grad = torch.empty_like(h_models[0]).pin_memory()
    h_row = torch.empty(rows, dtype=torch.float32).pin_memory()
    h_loss = torch.empty(1, dtype=torch.float32).pin_memory()
    h_cnt = torch.empty(3 + n - 1, dtype=torch.int64).pin_memory()
    h_st = torch.empty(1, dtype=torch.int32).pin_memory()
    dt_code = cb.dtype_code(models[0].dtype)
    ws = torch.empty(cb.host_workspace_bytes(n, rows, C, dt_code, 0), dtype=torch.uint8, device="cuda")
    ptrs = (ctypes.c_void_p * max(1, n - 1))(*[m.data_ptr() for m in h_models[1:]])
    p = cb.Params()
    p.struct_bytes = ctypes.sizeof(cb.Params)
    p.logits, p.peer_logits = h_models[0].data_ptr(), ctypes.cast(ptrs, ctypes.POINTER(ctypes.c_void_p))
    p.labels, p.mask = h_labels.data_ptr(), (h_mask.data_ptr() if h_mask is not None else None)
    p.n, p.dtype, p.rows, p.classes, p.row_stride = n, dt_code, rows, C, C
    p.alpha, p.temperature, p.label_smoothing = w.alpha, w.temperature, w.label_smoothing
    p.dist_kind = dist_code
    p.row_loss, p.reduced_loss, p.grad_logits = h_row.data_ptr(), h_loss.data_ptr(), h_grad.data_ptr()
    p.counters, p.dev_status = h_cnt.data_ptr(), h_st.data_ptr()
    p.workspace, p.workspace_bytes = ws.data_ptr(), ws.numel()
    stream = torch.cuda.current_stream()
    cb.codistill_loss_fwd_bwd_host(p, 0, stream)      # warm-up
    barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    for _ in range(args.e2e_steps):
        cb.codistill_loss_fwd_bwd_host(p, 0, stream)
    ev1.record(stream)
    barrier()
    ms = ev0.elapsed_time(ev1) / args.e2e_steps
    if world > 1:
        import torch.distributed as dist_pkg
        t = torch.tensor([ms], device="cuda", dtype=torch.float64)
        dist_pkg.all_reduce(t, op=dist_pkg.ReduceOp.MAX)
        ms = float(t.item())
    es = models[0].element_size()
    h2d = n * rows * C * es + rows * 4 + (rows if mask is not None else 0)
    d2h = rows * C * es + rows * 4 + 4 + 4 + 8 * (3 + n - 1)
    return {"value": world * rows / (ms * 1e-3), "unit": UNIT, "ms_per_step": ms, "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "steps": args.e2e_steps,
            "api": "codistill_loss_fwd_bwd_host (pinned host buffers, copies inside the timed region)"}


def torchrun_command(argv, gpus, port=None):
    """The command that runs this script as one process per GPU of this node."""
    if port is None:
        import socket
        with socket.socket() as s:
            s.bind(("127.0.0.1", 0))
            port = s.getsockname()[1]
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={gpus}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *argv]


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # asked for N GPUs outside a launcher: start one rank per GPU and let rank 0 print the line
        os.execvp(sys.executable, torchrun_command(sys.argv[1:], args.gpus))
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
