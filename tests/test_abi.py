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
                 "moesched_strerror", "moesched_status_str", "moesched_workspace_bytes", "moesched_last_cuda_error"):
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


def test_workspace_size_and_texts(lib):
    lib.moesched_workspace_bytes.restype = ctypes.c_size_t
    lib.moesched_status_str.restype = ctypes.c_char_p
    lib.moesched_strerror.restype = ctypes.c_char_p
    for B, N in ((1, 17), (4096, 64), (256, 256)):
        assert lib.moesched_workspace_bytes(B, N, 64) == lib.moesched_bvn_scratch_bytes(B, N) > 0
    assert lib.moesched_workspace_bytes(4, 300, 8) == 0 and lib.moesched_workspace_bytes(4, 64, 0) == 0
    # return codes and statuses share the numbers -1 and -2; each has its own text
    codes = {c: lib.moesched_strerror(c) for c in (0, -1, -2, -3)}
    stats = {c: lib.moesched_status_str(c) for c in (0, 1, -1, -2)}
    assert len(set(codes.values())) == 4 and len(set(stats.values())) == 4
    assert b"argument" in codes[-1] and b"CUDA" in codes[-2] and b"scratch" in codes[-3]
    assert b"input" in stats[-1] and b"limit" in stats[-2] and b"budget" in stats[1]
    assert codes[-1] != stats[-1] and codes[-2] != stats[-2]
    assert b"unknown" in lib.moesched_strerror(7) and b"unknown" in lib.moesched_status_str(7)


def test_header_is_valid_c99_and_the_binding_mirrors_its_struct(tmp_path):
    """The header must compile as plain C, and the ctypes struct of the binding restates
    moesched_model_t by hand: size, field order and offsets are checked against the compiler's."""
    import subprocess
    import paper_2605_26845_b200 as ms
    fields = [name for name, _ in ms._Model._fields_]
    prog = tmp_path / "abi.c"
    prog.write_text(
        '#include <stdio.h>\n#include <stddef.h>\n#include "moesched.h"\n'
        "int main(void) {\n"
        '  printf("%zu\\n", sizeof(moesched_model_t));\n'
        + "".join(f'  printf("%zu\\n", offsetof(moesched_model_t, {f}));\n' for f in fields)
        + '  printf("%d %d %d %d\\n", MOESCHED_OK, MOESCHED_EINVAL, MOESCHED_ECUDA, MOESCHED_ETOOBIG);\n'
        '  printf("%d %d %d %d\\n", MOESCHED_ST_OK, MOESCHED_ST_TRUNCATED, MOESCHED_ST_BAD_INPUT, MOESCHED_ST_INTERNAL);\n'
        '  printf("%d %u\\n", MOESCHED_WORK_FIELDS, MOESCHED_STATIC_SCRATCH_BYTES);\n'
        "  return 0;\n}\n")
    exe = tmp_path / "abi"
    subprocess.run(["gcc", "-std=c99", "-pedantic", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"),
                    str(prog), "-o", str(exe)], check=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split("\n")
    assert int(out[0]) == ctypes.sizeof(ms._Model) == 48
    for k, f in enumerate(fields):
        assert int(out[1 + k]) == getattr(ms._Model, f).offset
    n = 1 + len(fields)
    assert out[n].split() == ["0", "-1", "-2", "-3"]
    assert [int(v) for v in out[n + 1].split()] == [ms.ST_OK, ms.ST_TRUNCATED, ms.ST_BAD_INPUT, ms.ST_INTERNAL]
    assert [int(v) for v in out[n + 2].split()] == [ms.WORK_FIELDS, ms.STATIC_SCRATCH_BYTES]


def test_python_binding_refuses_cpu_tensors():
    import torch
    import paper_2605_26845_b200 as ms
    with pytest.raises(ms.MoeschedError):
        ms.mw_decompose(torch.zeros((1, 8, 8), dtype=torch.int32), 4)
