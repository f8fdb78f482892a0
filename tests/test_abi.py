"""The C-ABI library loads without a GPU and exports every symbol its header declares."""
import ctypes
import os
import re

import pytest

import __graft_entry__ as entry

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "moesched.h")


@pytest.fixture(scope="module")
def lib():
    entry.build()
    import paper_2605_26845_b200 as ms
    return ms.load_library()


def declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(moesched_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_entry_points():
    names = declared_functions()
    for want in ("moesched_mw_decompose", "moesched_bvn_decompose", "moesched_schedule_eval", "moesched_ideal_a2a", "moesched_schedule_prefix_eval",
                 "moesched_strerror", "moesched_last_cuda_error"):
        assert want in names


def test_every_declared_symbol_is_exported(lib):
    for name in declared_functions():
        assert hasattr(lib, name), name


def test_argument_validation_needs_no_gpu(lib):
    # invalid sizes and null pointers are rejected before any CUDA call
    null = ctypes.c_void_p(None)
    assert lib.moesched_mw_decompose(1, 0, null, 1, null, null, null, null, null, null, null) == -1
    assert lib.moesched_mw_decompose(1, 8, null, 1, null, null, null, null, null, null, null) == -1
    assert lib.moesched_bvn_decompose(1, 257, null, 1, null, null, null, null, null, null, null, null) == -1
    assert lib.moesched_bvn_scratch_bytes(2, 64) == 2 * 64 * 64 * 4
    assert lib.moesched_bvn_scratch_bytes(1, 17) == 17 * 24 * 4
    assert lib.moesched_bvn_scratch_bytes(1, 300) == 0
    assert lib.moesched_schedule_eval(1, 8, null, 1, null, null, null, null, null, null, null, null, null,
                                      null, null) == -1
    assert lib.moesched_ideal_a2a(1, 8, null, null, null, null, null, null) == -1
    assert lib.moesched_strerror(0) == b"ok"
    assert lib.moesched_last_cuda_error() == 0


def test_python_binding_refuses_cpu_tensors():
    import torch
    import paper_2605_26845_b200 as ms
    with pytest.raises(ms.MoeschedError):
        ms.mw_decompose(torch.zeros((1, 8, 8), dtype=torch.int32), 4)
