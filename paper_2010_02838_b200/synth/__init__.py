"""Seeded synthetic inputs shaped like the paper's workloads (host side, numpy).

This module holds none of the objective's arithmetic.  It serves the tests, the benchmark and
the CPU oracle alike: every tensor is a pure function of (seed, stream, element index), produced
by ``synth.c`` (SplitMix64 finaliser + Box-Muller), so any row slice can be regenerated alone.

The five workloads stand in for logits of the paper's image-classification heads (CIFAR-10,
ImageNet / ResNet-50) and translation heads (vocabulary 32K) -- Sections 4-5 and the appendix
"Implementation Details" -- whose datasets and trained models are not needed for this path.
bf16 tensors are returned as ``numpy.uint16`` bit patterns (round-to-nearest-even from fp32).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "synth.c")
_SO = os.path.join(_HERE, "libsynth.so")
_lib = None

STREAM_BASE, STREAM_LABELS, STREAM_MASK, STREAM_MODEL0 = 1, 2, 3, 16


def build(force: bool = False) -> str:
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        subprocess.run(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-Wall", "-o", _SO, _SRC, "-lm"], check=True)
    return _SO


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_SO)
        u64 = ctypes.c_uint64
        lib.synth_normal_f32.argtypes = [u64, u64, u64, u64, ctypes.c_void_p]
        lib.synth_uniform_i32.argtypes = [u64, u64, u64, u64, ctypes.c_int32, ctypes.c_void_p]
        lib.synth_raw_u64.argtypes = [u64, u64, u64, u64, ctypes.c_void_p]
        for f in (lib.synth_normal_f32, lib.synth_uniform_i32, lib.synth_raw_u64):
            f.restype = None
        _lib = lib
    return _lib


def normal_f32(seed: int, stream: int, first: int, count: int) -> np.ndarray:
    out = np.empty(count, dtype=np.float32)
    _load().synth_normal_f32(seed, stream, first, count, out.ctypes.data)
    return out


def uniform_i32(seed: int, stream: int, first: int, count: int, bound: int) -> np.ndarray:
    out = np.empty(count, dtype=np.int32)
    _load().synth_uniform_i32(seed, stream, first, count, bound, out.ctypes.data)
    return out


def raw_u64(seed: int, stream: int, first: int, count: int) -> np.ndarray:
    out = np.empty(count, dtype=np.uint64)
    _load().synth_raw_u64(seed, stream, first, count, out.ctypes.data)
    return out


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16, returned as uint16 bit patterns (finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    return ((u + (((u >> 16) & 1) + 0x7FFF)) >> 16).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << 16).view(np.float32)


@dataclass(frozen=True)
class Workload:
    """One synthetic workload.  ``kind``: 'indep' (models i.i.d.), 'own_plus_noise'
    (peer = own + noise) or 'shared_base' (every model = base + per-model noise)."""
    name: str
    n: int
    rows: int
    classes: int
    dtype: str            # 'f32' | 'bf16'
    kind: str
    sigma: float          # std of own / base
    sigma_noise: float    # std of the per-model noise (0 for 'indep')
    alpha: float
    temperature: float
    label_smoothing: float
    tokens_per_seq: int   # 0 = no padding mask
    n_padded: int         # exact number of masked rows
    seed: int = 0

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2

    def algorithmic_bytes(self, skip_masked_reads: bool = False) -> int:
        """(n+1)*R*C*s + 9R; with masked-row reads skipped: n*R_valid*C*s + R*C*s + 9R."""
        R, C, s, n = self.rows, self.classes, self.elem_bytes, self.n
        if skip_masked_reads:
            return n * (R - self.n_padded) * C * s + R * C * s + 9 * R
        return (n + 1) * R * C * s + 9 * R


WORKLOADS = {
    1: Workload("cifar10_head_n2", 2, 128, 10, "f32", "indep", 3.0, 0.0, 1.0, 1.0, 0.0, 0, 0),
    2: Workload("imagenet_head_n2", 2, 256, 1000, "f32", "own_plus_noise", 2.0, 0.5, 1.0, 1.0, 0.0, 0, 0),
    3: Workload("imagenet_head_n4_bf16", 4, 1024, 1000, "bf16", "shared_base", 2.0, 1.0, 0.5, 2.0, 0.0, 0, 0),
    4: Workload("translation_head_32k_n2_bf16", 2, 8192, 32768, "bf16", "indep", 1.5, 0.0, 1.0, 1.0, 0.1, 32, 819),
    5: Workload("lm_head_50257_n8_bf16", 8, 16384, 50257, "bf16", "shared_base", 1.5, 0.7, 1.0, 1.0, 0.0, 32, 819),
}


def scaled(w: Workload, rows: int | None = None, classes: int | None = None, name: str | None = None) -> Workload:
    """A smaller workload of the same recipe (padding fraction kept)."""
    import dataclasses
    R = w.rows if rows is None else rows
    pad = 0 if w.tokens_per_seq == 0 else max(1, round(w.n_padded * R / w.rows))
    return dataclasses.replace(w, rows=R, classes=w.classes if classes is None else classes,
                               n_padded=pad, name=name or f"{w.name}_r{R}")


def make_labels(w: Workload, row_begin: int = 0, row_end: int | None = None) -> np.ndarray:
    row_end = w.rows if row_end is None else row_end
    return uniform_i32(w.seed, STREAM_LABELS, row_begin, row_end - row_begin, w.classes)


def make_mask(w: Workload) -> np.ndarray | None:
    """1 = valid token.  Padding sits at the end of each sequence: every sequence gets
    floor(n_padded / n_seq) trailing pads and the first (n_padded mod n_seq) sequences of a seeded
    permutation get one more."""
    if w.tokens_per_seq == 0:
        return None
    L = w.tokens_per_seq
    n_seq = w.rows // L
    assert n_seq * L == w.rows
    per, extra = divmod(w.n_padded, n_seq)
    pads = np.full(n_seq, per, dtype=np.int64)
    order = np.argsort(raw_u64(w.seed, STREAM_MASK, 0, n_seq), kind="stable")
    pads[order[:extra]] += 1
    assert pads.max() <= L
    pos = np.arange(L)[None, :]
    mask = (pos < (L - pads)[:, None]).astype(np.uint8).reshape(-1)
    assert int((mask == 0).sum()) == w.n_padded
    return mask


def make_model_logits(w: Workload, k: int, row_begin: int = 0, row_end: int | None = None) -> np.ndarray:
    """Logits of model k (0 = own, 1..n-1 = peers) for rows [row_begin, row_end): [rows, classes],
    float32 or uint16 (bf16 bits).  Values are formed in fp32 and rounded once."""
    row_end = w.rows if row_end is None else row_end
    first, count = row_begin * w.classes, (row_end - row_begin) * w.classes
    sig, sn = np.float32(w.sigma), np.float32(w.sigma_noise)
    if w.kind == "indep":
        x = sig * normal_f32(w.seed, STREAM_MODEL0 + k, first, count)
    elif w.kind == "own_plus_noise":
        x = sig * normal_f32(w.seed, STREAM_MODEL0, first, count)
        if k > 0:
            x = x + sn * normal_f32(w.seed, STREAM_MODEL0 + k, first, count)
    elif w.kind == "shared_base":
        x = sig * normal_f32(w.seed, STREAM_BASE, first, count) + sn * normal_f32(w.seed, STREAM_MODEL0 + k, first, count)
    else:
        raise ValueError(w.kind)
    x = x.reshape(row_end - row_begin, w.classes)
    return x if w.dtype == "f32" else f32_to_bf16_bits(x)


def make_inputs(w: Workload, row_begin: int = 0, row_end: int | None = None):
    """(own, [peers], labels, mask-or-None) for a row range (mask sliced from the full mask)."""
    row_end = w.rows if row_end is None else row_end
    own = make_model_logits(w, 0, row_begin, row_end)
    peers = [make_model_logits(w, k, row_begin, row_end) for k in range(1, w.n)]
    labels = make_labels(w, row_begin, row_end)
    mask = make_mask(w)
    if mask is not None:
        mask = np.ascontiguousarray(mask[row_begin:row_end])
    return own, peers, labels, mask
