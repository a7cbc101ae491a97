"""TEST INFRASTRUCTURE -- double-precision CPU oracle of the codistillation objective.

Only ``tests/``, ``__graft_entry__.smoke()`` and the CPU-baseline / reference legs of ``bench.py``
may import this package.  It wraps ``codistill_oracle.c`` (plain C, fp64, OpenMP over rows only)
through ctypes with numpy arrays; it imports nothing from the CUDA package.

bf16 tensors are passed as ``numpy.uint16`` arrays holding the raw bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "codistill_oracle.c")
_SO = os.path.join(_HERE, "liboracle.so")

F32, BF16 = 0, 1
DIST_MSE, DIST_KL, DIST_MSE_CENTRED, DIST_KL_REVERSE, DIST_KL_SYMMETRIC = 0, 1, 2, 3, 4
PEERS_PAIRWISE, PEERS_MEAN_TARGET = 0, 1
REDUCE_MEAN_VALID, REDUCE_SUM = 0, 1

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math: the arithmetic must stay as written)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-Wall", "-Wextra", "-o", _SO, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _SO


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_SO)
        lib.codistill_oracle.restype = ctypes.c_int
        lib.codistill_oracle.argtypes = [
            ctypes.c_void_p, ctypes.POINTER(ctypes.c_void_p), ctypes.c_void_p, ctypes.c_void_p,
            ctypes.c_int, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, ctypes.c_int,
            ctypes.c_double, ctypes.c_double, ctypes.c_double, ctypes.c_int, ctypes.c_int, ctypes.c_int,
            ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int,
        ]
        lib.codistill_oracle_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def max_threads() -> int:
    return int(_load().codistill_oracle_threads())


@dataclass
class OracleResult:
    row_loss: np.ndarray      # [rows] float64, unscaled per-row loss (0 for masked rows)
    loss: float               # reduced loss
    grad: np.ndarray | None   # [grad_end - grad_begin, classes] float64
    counters: np.ndarray      # [3 + (n-1)] int64: n_valid, n_masked, n_correct, n_agree[j]
    status: int


def _dtype_code(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.uint16:
        return BF16
    raise TypeError(f"logits must be float32 or uint16 (bf16 bits), got {a.dtype}")


def codistill(own: np.ndarray, peers, labels: np.ndarray, mask: np.ndarray | None = None, *,
              classes: int | None = None, alpha: float = 1.0, temperature: float = 1.0,
              label_smoothing: float = 0.0, dist: int = DIST_MSE, peer_reduce: int = PEERS_PAIRWISE,
              reduction: int = REDUCE_MEAN_VALID, want_grad: bool = True, grad_rows=None,
              nthreads: int = 0) -> OracleResult:
    """Evaluate the objective for one model.  ``own`` is [rows, row_stride]; ``classes`` defaults
    to the row pitch.  ``grad_rows=(begin, end)`` restricts the rows whose gradient is returned."""
    lib = _load()
    assert own.ndim == 2 and own.flags.c_contiguous
    rows, stride = own.shape
    C = stride if classes is None else int(classes)
    dt = _dtype_code(own)
    peers = list(peers)
    n = len(peers) + 1
    for p in peers:
        assert p.shape == own.shape and p.dtype == own.dtype and p.flags.c_contiguous
    labels = np.ascontiguousarray(labels, dtype=np.int32)
    assert labels.shape == (rows,)
    if mask is not None:
        mask = np.ascontiguousarray(mask, dtype=np.uint8)
        assert mask.shape == (rows,)
    ptrs = (ctypes.c_void_p * max(1, len(peers)))(*[p.ctypes.data for p in peers])
    gb, ge = (0, rows) if grad_rows is None else (int(grad_rows[0]), int(grad_rows[1]))
    grad = np.empty((ge - gb, C), dtype=np.float64) if want_grad else None
    row_loss = np.zeros(rows, dtype=np.float64)
    loss = np.zeros(1, dtype=np.float64)
    counters = np.zeros(3 + (n - 1), dtype=np.int64)
    status = np.zeros(1, dtype=np.int32)
    rc = lib.codistill_oracle(
        own.ctypes.data if rows else None, ptrs, labels.ctypes.data if rows else None,
        mask.ctypes.data if (mask is not None and rows) else None,
        n, rows, C, stride, dt, float(alpha), float(temperature), float(label_smoothing),
        int(dist), int(peer_reduce), int(reduction), gb, ge,
        row_loss.ctypes.data, loss.ctypes.data, grad.ctypes.data if want_grad else None,
        counters.ctypes.data, status.ctypes.data, int(nthreads))
    if rc != 0:
        raise ValueError("codistill_oracle: invalid arguments")
    return OracleResult(row_loss, float(loss[0]), grad, counters, int(status[0]))


def codistill_all(models, labels: np.ndarray, mask: np.ndarray | None = None, **options):
    """Algorithm 1's inner loop "for i = 1..n": the objective of every model i with the other models,
    in increasing index, as its peers.  Written out as n evaluations of the single-model definition;
    returns the list of their results."""
    models = list(models)
    return [codistill(models[i], models[:i] + models[i + 1:], labels, mask, **options) for i in range(len(models))]
