"""The C-ABI library builds, loads and exports every symbol declared in include/*.h
(no compute calls: runs without a GPU)."""
import ctypes
import os
import re

import pytest

from paper_2010_02838_b200 import binding as cb
from paper_2010_02838_b200 import build as cbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    cbuild.build()
    return cb.load_library()


def declared_functions():
    names = set()
    inc = os.path.join(ROOT, "include")
    for header in sorted(os.listdir(inc)):
        text = open(os.path.join(inc, header)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b(codistill_[a-z_0-9]+)\s*\(", text))
    return sorted(names)


def test_exports_every_declared_symbol(lib):
    names = declared_functions()
    assert set(names) == set(cb.EXPORTS)
    for name in names:
        assert getattr(lib, name) is not None


def test_params_struct_matches_header(lib):
    # field order and size of the ctypes mirror follow the header's struct
    text = open(os.path.join(ROOT, "include", "codistill.h")).read()
    body = text[text.index("typedef struct codistill_params {"):text.index("} codistill_params_t;")]
    fields = re.findall(r"\b([a-z_]+);", body)
    assert fields == [f[0] for f in cb.Params._fields_]
    assert ctypes.sizeof(cb.Params) == 152  # static_assert-ed on the C side


def test_host_side_queries(lib):
    assert cb.version() >= 100
    assert cb.status_string(0) == "ok" and "workspace" in cb.status_string(7)
    ws = cb.workspace_bytes(2, 8192, 32768, cb.BF16)
    assert ws % 256 == 0 and ws >= 256 + 8192 * 8
    assert cb.host_workspace_bytes(2, 8192, 32768, cb.BF16, 512) > ws + 2 * 3 * 512 * 32768 * 2 - 1


def test_argument_validation_needs_no_gpu(lib):
    p = cb.Params()
    p.struct_bytes = ctypes.sizeof(cb.Params)
    assert lib.codistill_loss_fwd_bwd_ex(None, None) == 1
    p.n, p.rows, p.classes, p.row_stride, p.temperature = 0, 4, 8, 8, 1.0
    assert lib.codistill_loss_fwd_bwd_ex(ctypes.byref(p), None) == 2       # n < 1
    p.n, p.row_stride = 2, 4
    assert lib.codistill_loss_fwd_bwd_ex(ctypes.byref(p), None) == 2       # pitch < classes
    p.row_stride, p.dtype = 8, 7
    assert lib.codistill_loss_fwd_bwd_ex(ctypes.byref(p), None) == 3       # dtype
    p.dtype, p.temperature = 0, 0.0
    assert lib.codistill_loss_fwd_bwd_ex(ctypes.byref(p), None) == 4       # temperature
    p.temperature, p.label_smoothing = 1.0, 1.0
    assert lib.codistill_loss_fwd_bwd_ex(ctypes.byref(p), None) == 4       # label smoothing
    p.label_smoothing, p.alpha = 0.0, float("inf")
    assert lib.codistill_loss_fwd_bwd_ex(ctypes.byref(p), None) == 4       # alpha
    p.alpha, p.n = 1.0, 40
    assert lib.codistill_loss_fwd_bwd_ex(ctypes.byref(p), None) == 5       # too many peers
    p.n = 2
    assert lib.codistill_loss_fwd_bwd_ex(ctypes.byref(p), None) == 1       # reduced_loss NULL
    p.struct_bytes = 8
    assert lib.codistill_loss_fwd_bwd_ex(ctypes.byref(p), None) == 4       # ABI size mismatch


def test_binding_refuses_cpu_tensors(lib):
    import torch
    x = torch.zeros(4, 8)
    with pytest.raises(ValueError):
        cb.codistill_loss_fwd_bwd(x, [x], torch.zeros(4, dtype=torch.int32))
