"""Thin ctypes binding over ``libcodistill.so`` (see ``include/codistill.h``).

Argument marshalling only: every step of the objective runs in the CUDA kernels.  PyTorch is
used for device memory and streams.  There is no CPU fallback: if the library is missing or the
tensors are not on a CUDA device the calls raise.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcodistill.so")

OK = 0
F32, BF16 = 0, 1
DIST_MSE_LOGITS, DIST_KL_SOFTMAX, DIST_MSE_CENTRED, DIST_KL_REVERSE, DIST_KL_SYMMETRIC = 0, 1, 2, 3, 4
PEERS_PAIRWISE_MEAN, PEERS_MEAN_TARGET = 0, 1
REDUCE_MEAN_VALID, REDUCE_SUM = 0, 1
DEV_BAD_LABEL, DEV_TIMEOUT = 1, 2
MAX_PEERS = 31
STATIC_MAX_ROWS = 65536
ERR_CUDA = 6
ERR_TOO_LARGE = 8

EXPORTS = (
    "codistill_loss_fwd_bwd", "codistill_loss_fwd_bwd_ex", "codistill_loss_fwd_bwd_host",
    "codistill_loss_fwd_bwd_static", "codistill_loss_fwd_bwd_all", "codistill_all_workspace_bytes",
    "codistill_workspace_bytes", "codistill_host_workspace_bytes", "codistill_status_string",
    "codistill_version", "codistill_kernel_regime", "codistill_last_cuda_error",
    "codistill_selftest_bounded_wait", "codistill_pack_predictions", "codistill_unpack_predictions",
    "codistill_schedule_alpha", "codistill_schedule_piecewise", "codistill_schedule_step_decay",
    "codistill_is_exchange_step", "codistill_bits_all_reduce", "codistill_bits_checkpoints",
    "codistill_bits_predictions",
)


class Params(ctypes.Structure):
    """Mirror of ``codistill_params_t``."""
    _fields_ = [
        ("struct_bytes", ctypes.c_uint64),
        ("logits", ctypes.c_void_p),
        ("peer_logits", ctypes.POINTER(ctypes.c_void_p)),
        ("labels", ctypes.c_void_p),
        ("mask", ctypes.c_void_p),
        ("n", ctypes.c_int32),
        ("dtype", ctypes.c_int32),
        ("rows", ctypes.c_int64),
        ("classes", ctypes.c_int64),
        ("row_stride", ctypes.c_int64),
        ("alpha", ctypes.c_float),
        ("temperature", ctypes.c_float),
        ("label_smoothing", ctypes.c_float),
        ("dist_kind", ctypes.c_int32),
        ("peer_reduce", ctypes.c_int32),
        ("reduction", ctypes.c_int32),
        ("row_loss", ctypes.c_void_p),
        ("reduced_loss", ctypes.c_void_p),
        ("grad_logits", ctypes.c_void_p),
        ("counters", ctypes.c_void_p),
        ("dev_status", ctypes.c_void_p),
        ("workspace", ctypes.c_void_p),
        ("workspace_bytes", ctypes.c_uint64),
    ]


class AllParams(ctypes.Structure):
    """Mirror of ``codistill_all_params_t``."""
    _fields_ = [
        ("struct_bytes", ctypes.c_uint64),
        ("logits", ctypes.POINTER(ctypes.c_void_p)),
        ("labels", ctypes.c_void_p),
        ("mask", ctypes.c_void_p),
        ("n", ctypes.c_int32),
        ("dtype", ctypes.c_int32),
        ("rows", ctypes.c_int64),
        ("classes", ctypes.c_int64),
        ("row_stride", ctypes.c_int64),
        ("alpha", ctypes.c_float),
        ("label_smoothing", ctypes.c_float),
        ("peer_reduce", ctypes.c_int32),
        ("reduction", ctypes.c_int32),
        ("dist_kind", ctypes.c_int32),
        ("temperature", ctypes.c_float),
        ("row_loss", ctypes.c_void_p),
        ("reduced_loss", ctypes.c_void_p),
        ("grad_logits", ctypes.POINTER(ctypes.c_void_p)),
        ("counters", ctypes.c_void_p),
        ("dev_status", ctypes.c_void_p),
        ("workspace", ctypes.c_void_p),
        ("workspace_bytes", ctypes.c_uint64),
    ]


class CodistillError(RuntimeError):
    def __init__(self, code: int):
        self.code = code
        detail = f" ({load_library().codistill_last_cuda_error().decode()})" if code == ERR_CUDA else ""
        super().__init__(f"codistill error {code}: {status_string(code)}{detail}")


_lib = None


def load_library() -> ctypes.CDLL:
    """Load the C-ABI library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is not None:
        return _lib
    path = os.environ.get("CODISTILL_LIBRARY", LIB_PATH)   # another build of the same library (same ABI), e.g. for A/B timing
    if not os.path.exists(path):
        raise RuntimeError(
            f"{path} is missing: build it with `python -m paper_2010_02838_b200.build` "
            "(nvcc, sm_100a). There is no CPU or PyTorch fallback for the codistillation kernels.")
    lib = ctypes.CDLL(path)
    vp, i64, i32, f32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_float
    lib.codistill_loss_fwd_bwd.restype = i32
    lib.codistill_loss_fwd_bwd.argtypes = [vp, ctypes.POINTER(vp), vp, vp, i32, i64, i64, f32, f32, i32, vp, vp, vp, vp]
    lib.codistill_loss_fwd_bwd_static.restype = i32
    lib.codistill_loss_fwd_bwd_static.argtypes = lib.codistill_loss_fwd_bwd.argtypes
    lib.codistill_loss_fwd_bwd_ex.restype = i32
    lib.codistill_loss_fwd_bwd_ex.argtypes = [ctypes.POINTER(Params), vp]
    lib.codistill_loss_fwd_bwd_host.restype = i32
    lib.codistill_loss_fwd_bwd_host.argtypes = [ctypes.POINTER(Params), i64, vp]
    lib.codistill_loss_fwd_bwd_all.restype = i32
    lib.codistill_loss_fwd_bwd_all.argtypes = [ctypes.POINTER(AllParams), vp]
    lib.codistill_all_workspace_bytes.restype = ctypes.c_size_t
    lib.codistill_all_workspace_bytes.argtypes = [i32, i64]
    lib.codistill_workspace_bytes.restype = ctypes.c_size_t
    lib.codistill_workspace_bytes.argtypes = [i32, i64, i64, i32]
    lib.codistill_host_workspace_bytes.restype = ctypes.c_size_t
    lib.codistill_host_workspace_bytes.argtypes = [i32, i64, i64, i32, i64]
    lib.codistill_status_string.restype = ctypes.c_char_p
    lib.codistill_status_string.argtypes = [i32]
    for fn in (lib.codistill_pack_predictions, lib.codistill_unpack_predictions):
        fn.restype = i32
        fn.argtypes = [vp, vp, i64, i64, i64, i64, vp]
    lib.codistill_selftest_bounded_wait.restype = i32
    lib.codistill_selftest_bounded_wait.argtypes = [vp, ctypes.c_uint64, vp]
    lib.codistill_last_cuda_error.restype = ctypes.c_char_p
    lib.codistill_last_cuda_error.argtypes = []
    lib.codistill_version.restype = i32
    lib.codistill_version.argtypes = []
    lib.codistill_kernel_regime.restype = ctypes.c_char_p
    lib.codistill_kernel_regime.argtypes = [i32, i64, i64, i64, i32, i32, i32]
    f64, pd, pi64 = ctypes.c_double, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_int64)
    lib.codistill_schedule_alpha.restype = f64
    lib.codistill_schedule_alpha.argtypes = [f64, f64, i64]
    lib.codistill_schedule_piecewise.restype = f64
    lib.codistill_schedule_piecewise.argtypes = [pd, pi64, i32, i64]
    lib.codistill_schedule_step_decay.restype = f64
    lib.codistill_schedule_step_decay.argtypes = [f64, f64, pi64, i32, i64]
    lib.codistill_is_exchange_step.restype = i32
    lib.codistill_is_exchange_step.argtypes = [i64, i64]
    lib.codistill_bits_all_reduce.restype = f64
    lib.codistill_bits_all_reduce.argtypes = [f64]
    lib.codistill_bits_checkpoints.restype = f64
    lib.codistill_bits_checkpoints.argtypes = [i32, f64, i64]
    lib.codistill_bits_predictions.restype = f64
    lib.codistill_bits_predictions.argtypes = [i32, i64, i32, i64, i64]
    _lib = lib
    return lib


def status_string(code: int) -> str:
    return load_library().codistill_status_string(code).decode()


def version() -> int:
    return int(load_library().codistill_version())


def dtype_code(t: torch.dtype) -> int:
    if t == torch.float32:
        return F32
    if t == torch.bfloat16:
        return BF16
    raise TypeError(f"logits must be float32 or bfloat16, got {t}")


def workspace_bytes(n: int, rows: int, classes: int, dtype: int) -> int:
    return int(load_library().codistill_workspace_bytes(n, rows, classes, dtype))


def host_workspace_bytes(n: int, rows: int, classes: int, dtype: int, chunk_rows: int = 0) -> int:
    return int(load_library().codistill_host_workspace_bytes(n, rows, classes, dtype, chunk_rows))


def kernel_regime(n: int, rows: int, classes: int, row_stride: int | None = None, dtype: int = BF16,
                  dist: int = DIST_MSE_LOGITS, peer_reduce: int = PEERS_PAIRWISE_MEAN) -> str:
    r = load_library().codistill_kernel_regime(n, rows, classes, classes if row_stride is None else row_stride,
                                               dtype, dist, peer_reduce)
    return r.decode() if r else ""


@dataclass
class Outputs:
    """Device tensors written by one call (valid after the stream is synchronised)."""
    row_loss: torch.Tensor | None
    loss: torch.Tensor            # [1] float32
    grad: torch.Tensor | None     # like logits
    counters: torch.Tensor | None  # [3 + (n-1)] int64
    status: torch.Tensor | None   # [1] int32


def _ptr(t: torch.Tensor | None):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream_ptr(stream: torch.cuda.Stream | None):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _require_cuda(*tensors):
    for t in tensors:
        if t is not None and not t.is_cuda:
            raise ValueError("codistill kernels need CUDA tensors; there is no CPU path")


def _check_shapes(logits, peers, labels, mask, classes):
    if logits.dim() != 2 or logits.stride(1) != 1:
        raise ValueError("logits must be [rows, >=classes] with unit inner stride")
    rows, stride = logits.shape[0], (logits.stride(0) if logits.shape[0] > 1 else max(logits.stride(0), logits.shape[1]))
    C = logits.shape[1] if classes is None else int(classes)
    for p in peers:
        if p.shape != logits.shape or p.dtype != logits.dtype or p.stride() != logits.stride():
            raise ValueError("every peer must match logits in shape, dtype and strides")
    if labels.dtype != torch.int32 or labels.shape != (rows,) or not labels.is_contiguous():
        raise ValueError("labels must be a contiguous int32 [rows] tensor")
    if mask is not None and (mask.dtype != torch.uint8 or mask.shape != (rows,) or not mask.is_contiguous()):
        raise ValueError("mask must be a contiguous uint8 [rows] tensor")
    return rows, stride, C


def codistill_loss_fwd_bwd(logits: torch.Tensor, peer_logits, labels: torch.Tensor, mask: torch.Tensor | None = None,
                           *, alpha: float = 1.0, temperature: float = 1.0, want_row_loss: bool = True,
                           want_grad: bool = True, out: Outputs | None = None,
                           stream: torch.cuda.Stream | None = None) -> Outputs:
    """The call named ``codistill_loss_fwd_bwd`` in the C ABI: MSE-on-logits distance averaged over
    the peers, mean over valid rows, dense rows.  Returns device tensors (asynchronous)."""
    lib = load_library()
    peers = list(peer_logits)
    _require_cuda(logits, labels, mask, *peers)
    rows, stride, C = _check_shapes(logits, peers, labels, mask, None)
    if rows > 1 and stride != C:
        raise ValueError("the basic call needs dense rows; use codistill_loss_fwd_bwd_ex for a row pitch")
    if out is None:
        out = Outputs(
            torch.empty(rows, dtype=torch.float32, device=logits.device) if want_row_loss else None,
            torch.empty(1, dtype=torch.float32, device=logits.device),
            torch.empty_like(logits) if want_grad else None, None, None)
    ptrs = (ctypes.c_void_p * max(1, len(peers)))(*[p.data_ptr() for p in peers])
    rc = lib.codistill_loss_fwd_bwd(_ptr(logits), ptrs, _ptr(labels), _ptr(mask), len(peers) + 1, rows, C,
                                    float(alpha), float(temperature), dtype_code(logits.dtype),
                                    _ptr(out.row_loss), _ptr(out.loss), _ptr(out.grad), _stream_ptr(stream))
    if rc != OK:
        raise CodistillError(rc)
    return out


def codistill_loss_fwd_bwd_static(logits: torch.Tensor, peer_logits, labels: torch.Tensor,
                                  mask: torch.Tensor | None, out: Outputs, *, alpha: float = 1.0,
                                  temperature: float = 1.0, stream: torch.cuda.Stream | None = None) -> Outputs:
    """The allocation-free entry point of the C ABI.  For callers that must not touch a CUDA
    allocator at call time (all device memory already claimed by a framework, or a loop that bans
    allocator calls): the library's scratch is a fixed array in its device image, good for at most
    ``STATIC_MAX_ROWS`` rows.  Nothing is allocated here either, so ``out`` (loss, and optionally row_loss
    and grad) must be supplied.  Calls on one device share the scratch: keep them ordered."""
    lib = load_library()
    peers = list(peer_logits)
    _require_cuda(logits, labels, mask, out.row_loss, out.loss, out.grad, *peers)
    rows, stride, C = _check_shapes(logits, peers, labels, mask, None)
    if rows > 1 and stride != C:
        raise ValueError("the allocation-free call needs dense rows")
    ptrs = (ctypes.c_void_p * max(1, len(peers)))(*[p.data_ptr() for p in peers])
    rc = lib.codistill_loss_fwd_bwd_static(_ptr(logits), ptrs, _ptr(labels), _ptr(mask), len(peers) + 1, rows, C,
                                           float(alpha), float(temperature), dtype_code(logits.dtype),
                                           _ptr(out.row_loss), _ptr(out.loss), _ptr(out.grad), _stream_ptr(stream))
    if rc != OK:
        raise CodistillError(rc)
    return out


class Plan:
    """Pre-allocated outputs, workspace and parameter block for repeated ``_ex`` calls on one shape.
    ``run()`` does no allocation and no tensor bookkeeping: it only calls the C entry point."""

    def __init__(self, logits: torch.Tensor, peer_logits, labels: torch.Tensor, mask: torch.Tensor | None = None, *,
                 classes: int | None = None, alpha: float = 1.0, temperature: float = 1.0,
                 label_smoothing: float = 0.0, dist: int = DIST_MSE_LOGITS, peer_reduce: int = PEERS_PAIRWISE_MEAN,
                 reduction: int = REDUCE_MEAN_VALID, want_row_loss: bool = True, want_grad: bool = True,
                 want_counters: bool = True, workspace: torch.Tensor | None = None):
        self.lib = load_library()
        peers = list(peer_logits)
        _require_cuda(logits, labels, mask, *peers)
        rows, stride, C = _check_shapes(logits, peers, labels, mask, classes)
        n = len(peers) + 1
        dev = logits.device
        dt = dtype_code(logits.dtype)
        self.keep = (logits, peers, labels, mask)
        self.out = Outputs(
            torch.empty(rows, dtype=torch.float32, device=dev) if want_row_loss else None,
            torch.empty(1, dtype=torch.float32, device=dev),
            torch.empty_strided(logits.shape, logits.stride(), dtype=logits.dtype, device=dev) if want_grad else None,
            torch.empty(3 + n - 1, dtype=torch.int64, device=dev) if want_counters else None,
            torch.empty(1, dtype=torch.int32, device=dev))
        need = int(self.lib.codistill_workspace_bytes(n, rows, C, dt))
        self.workspace = workspace if workspace is not None else torch.empty(need, dtype=torch.uint8, device=dev)
        self.ptrs = (ctypes.c_void_p * max(1, len(peers)))(*[p.data_ptr() for p in peers])
        p = Params()
        p.struct_bytes = ctypes.sizeof(Params)
        p.logits = logits.data_ptr()
        p.peer_logits = ctypes.cast(self.ptrs, ctypes.POINTER(ctypes.c_void_p))
        p.labels = labels.data_ptr()
        p.mask = mask.data_ptr() if mask is not None else None
        p.n, p.dtype, p.rows, p.classes, p.row_stride = n, dt, rows, C, stride
        p.alpha, p.temperature, p.label_smoothing = float(alpha), float(temperature), float(label_smoothing)
        p.dist_kind, p.peer_reduce, p.reduction = int(dist), int(peer_reduce), int(reduction)
        p.row_loss = self.out.row_loss.data_ptr() if want_row_loss else None
        p.reduced_loss = self.out.loss.data_ptr()
        p.grad_logits = self.out.grad.data_ptr() if want_grad else None
        p.counters = self.out.counters.data_ptr() if want_counters else None
        p.dev_status = self.out.status.data_ptr()
        p.workspace = self.workspace.data_ptr()
        p.workspace_bytes = self.workspace.numel()
        self.params = p
        self.regime = kernel_regime(n, rows, C, stride, dt, dist, peer_reduce)

    def run(self, stream: torch.cuda.Stream | None = None) -> Outputs:
        rc = self.lib.codistill_loss_fwd_bwd_ex(ctypes.byref(self.params), _stream_ptr(stream))
        if rc != OK:
            raise CodistillError(rc)
        return self.out


def codistill_loss_fwd_bwd_ex(logits, peer_logits, labels, mask=None, stream=None, **options) -> Outputs:
    """One-shot form of :class:`Plan` (allocates outputs and workspace through PyTorch)."""
    return Plan(logits, peer_logits, labels, mask, **options).run(stream)


def codistill_loss_fwd_bwd_host(params: Params, chunk_rows: int = 0, stream: torch.cuda.Stream | None = None) -> None:
    """Host-buffer entry point; ``params`` holds HOST data pointers and a DEVICE workspace."""
    rc = load_library().codistill_loss_fwd_bwd_host(ctypes.byref(params), int(chunk_rows), _stream_ptr(stream))
    if rc != OK:
        raise CodistillError(rc)


@dataclass
class AllOutputs:
    """Device tensors written by one all-models call (valid after the stream is synchronised)."""
    row_loss: torch.Tensor        # [n, rows] float32
    loss: torch.Tensor            # [n] float32
    grads: list | None            # n tensors like the logits
    counters: torch.Tensor        # [n, 3 + (n-1)] int64
    status: torch.Tensor          # [1] int32


class AllPlan:
    """Pre-allocated outputs, workspace and parameter block for ``codistill_loss_fwd_bwd_all``: the
    objectives of all n models (each with the others as its peers) in one call."""

    def __init__(self, models, labels: torch.Tensor, mask: torch.Tensor | None = None, *, classes: int | None = None,
                 alpha: float = 1.0, temperature: float = 1.0, label_smoothing: float = 0.0,
                 dist: int = DIST_MSE_LOGITS, peer_reduce: int = PEERS_PAIRWISE_MEAN,
                 reduction: int = REDUCE_MEAN_VALID, want_grad: bool = True):
        self.lib = load_library()
        models = list(models)
        _require_cuda(labels, mask, *models)
        rows, stride, C = _check_shapes(models[0], models[1:], labels, mask, classes)
        n, dev, dt = len(models), models[0].device, dtype_code(models[0].dtype)
        self.keep = (models, labels, mask)
        grads = [torch.empty_strided(m.shape, m.stride(), dtype=m.dtype, device=dev) for m in models] if want_grad else None
        self.out = AllOutputs(torch.empty((n, rows), dtype=torch.float32, device=dev),
                              torch.empty(n, dtype=torch.float32, device=dev), grads,
                              torch.empty((n, 3 + n - 1), dtype=torch.int64, device=dev),
                              torch.empty(1, dtype=torch.int32, device=dev))
        need = int(self.lib.codistill_all_workspace_bytes(n, rows))
        self.workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)
        self.ptrs = (ctypes.c_void_p * n)(*[m.data_ptr() for m in models])
        self.gptrs = (ctypes.c_void_p * n)(*[g.data_ptr() for g in grads]) if want_grad else None
        p = AllParams()
        p.struct_bytes = ctypes.sizeof(AllParams)
        p.logits = ctypes.cast(self.ptrs, ctypes.POINTER(ctypes.c_void_p))
        p.labels = labels.data_ptr()
        p.mask = mask.data_ptr() if mask is not None else None
        p.n, p.dtype, p.rows, p.classes, p.row_stride = n, dt, rows, C, stride
        p.alpha, p.label_smoothing, p.temperature = float(alpha), float(label_smoothing), float(temperature)
        p.peer_reduce, p.reduction, p.dist_kind = int(peer_reduce), int(reduction), int(dist)
        p.row_loss = self.out.row_loss.data_ptr()
        p.reduced_loss = self.out.loss.data_ptr()
        p.grad_logits = ctypes.cast(self.gptrs, ctypes.POINTER(ctypes.c_void_p)) if want_grad else None
        p.counters = self.out.counters.data_ptr()
        p.dev_status = self.out.status.data_ptr()
        p.workspace = self.workspace.data_ptr()
        p.workspace_bytes = self.workspace.numel()
        self.params = p

    def run(self, stream: torch.cuda.Stream | None = None) -> AllOutputs:
        rc = self.lib.codistill_loss_fwd_bwd_all(ctypes.byref(self.params), _stream_ptr(stream))
        if rc != OK:
            raise CodistillError(rc)
        return self.out


def _rows_and_pitch(t: torch.Tensor):
    if t.dim() != 2 or (t.numel() > 0 and t.shape[1] > 1 and t.stride(1) != 1):
        raise ValueError("predictions must be [rows, classes] with unit inner stride")
    return t.shape[0], t.shape[1], (t.stride(0) if t.shape[0] > 1 else max(t.stride(0), t.shape[1]))


def pack_predictions(logits: torch.Tensor, out: torch.Tensor | None = None, stream: torch.cuda.Stream | None = None) -> torch.Tensor:
    """fp32 predictions -> bfloat16 (round to nearest even) on the device, for the exchange between model groups."""
    _require_cuda(logits, out)
    if logits.dtype != torch.float32:
        raise TypeError("pack_predictions takes float32 logits")
    rows, C, pitch = _rows_and_pitch(logits)
    if out is None:
        out = torch.empty((rows, C), dtype=torch.bfloat16, device=logits.device)
    orows, oC, opitch = _rows_and_pitch(out)
    if (orows, oC) != (rows, C) or out.dtype != torch.bfloat16:
        raise ValueError("out must be a bfloat16 tensor of the same shape")
    rc = load_library().codistill_pack_predictions(_ptr(logits), _ptr(out), rows, C, pitch, opitch, _stream_ptr(stream))
    if rc != OK:
        raise CodistillError(rc)
    return out


def unpack_predictions(packed: torch.Tensor, out: torch.Tensor | None = None, stream: torch.cuda.Stream | None = None) -> torch.Tensor:
    """bfloat16 predictions -> fp32 (exact) on the device."""
    _require_cuda(packed, out)
    if packed.dtype != torch.bfloat16:
        raise TypeError("unpack_predictions takes bfloat16 predictions")
    rows, C, pitch = _rows_and_pitch(packed)
    if out is None:
        out = torch.empty((rows, C), dtype=torch.float32, device=packed.device)
    orows, oC, opitch = _rows_and_pitch(out)
    if (orows, oC) != (rows, C) or out.dtype != torch.float32:
        raise ValueError("out must be a float32 tensor of the same shape")
    rc = load_library().codistill_unpack_predictions(_ptr(packed), _ptr(out), rows, C, pitch, opitch, _stream_ptr(stream))
    if rc != OK:
        raise CodistillError(rc)
    return out


def selftest_bounded_wait(limit_ns: int = 1_000_000, stream: torch.cuda.Stream | None = None) -> torch.Tensor:
    """Diagnostic: one CTA waits `limit_ns` on a barrier nothing completes; returns the [1] int32 status tensor."""
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rc = load_library().codistill_selftest_bounded_wait(_ptr(status), int(limit_ns), _stream_ptr(stream))
    if rc != OK:
        raise CodistillError(rc)
    return status


# ------------------------------------------------------------------ host-side schedules (codistill_schedule.h)
def schedule_alpha(alpha0: float, gamma: float, epoch: int) -> float:
    return float(load_library().codistill_schedule_alpha(float(alpha0), float(gamma), int(epoch)))


def _i64_array(xs):
    xs = [int(x) for x in xs]
    return (ctypes.c_int64 * max(1, len(xs)))(*xs), len(xs)


def schedule_piecewise(values, milestones, epoch: int) -> float:
    vals = (ctypes.c_double * len(values))(*[float(v) for v in values])
    ms, n = _i64_array(milestones)
    if len(values) != n + 1:
        raise ValueError("values must have one entry more than milestones")
    return float(load_library().codistill_schedule_piecewise(vals, ms, n, int(epoch)))


def schedule_step_decay(base: float, factor: float, milestones, epoch: int) -> float:
    ms, n = _i64_array(milestones)
    return float(load_library().codistill_schedule_step_decay(float(base), float(factor), ms, n, int(epoch)))


def is_exchange_step(step: int, period: int) -> bool:
    return bool(load_library().codistill_is_exchange_step(int(step), int(period)))


def bits_all_reduce(b_model: float) -> float:
    return float(load_library().codistill_bits_all_reduce(float(b_model)))


def bits_checkpoints(n: int, b_model: float, period: int) -> float:
    return float(load_library().codistill_bits_checkpoints(int(n), float(b_model), int(period)))


def bits_predictions(n: int, classes: int, bits_per_value: int, batch_per_device: int, period: int) -> float:
    return float(load_library().codistill_bits_predictions(int(n), int(classes), int(bits_per_value),
                                                           int(batch_per_device), int(period)))
