"""CPU-side checks of the C ABI: the library loads, exports every symbol the header declares, and its
host-side validation returns the documented codes.  No kernel is launched here."""
import ctypes as C
import os
import re

import pytest

from paper_2606_01813_b200 import binding as G
from paper_2606_01813_b200 import build as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    B.build()
    return G.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "cadd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cadd_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert set(names) == set(G.EXPORTS)
    for n in names:
        assert hasattr(lib, n), n


def test_struct_sizes_match_header(lib):
    # the library rejects a struct_size it was not built with, so a successful query proves both sides agree
    out = C.c_size_t()
    a = G.BuildArgs(); a.struct_size = C.sizeof(G.BuildArgs)
    a.batch, a.L, a.V, a.K, a.B_max, a.R = 4, 16, 151936, 8, 256, 257
    assert lib.cadd_build_workspace_bytes(C.byref(a), C.byref(out)) == G.OK and out.value > 0
    a.struct_size += 8
    assert lib.cadd_build_workspace_bytes(C.byref(a), C.byref(out)) == G.ERR_STRUCT_SIZE
    v = G.VerifyArgs(); v.struct_size = C.sizeof(G.VerifyArgs)
    v.batch, v.L, v.R, v.V = 4, 16, 257, 151936
    assert lib.cadd_verify_workspace_bytes(C.byref(v), C.byref(out)) == G.OK
    v.struct_size -= 4
    assert lib.cadd_verify_workspace_bytes(C.byref(v), C.byref(out)) == G.ERR_STRUCT_SIZE


def test_host_validation_codes(lib):
    out = C.c_size_t()
    assert lib.cadd_build_workspace_bytes(None, C.byref(out)) == G.ERR_NULL
    a = G.BuildArgs(); a.struct_size = C.sizeof(G.BuildArgs)
    a.batch, a.L, a.V, a.K, a.B_max, a.R = 1, 8, 1024, 4, 32, 33
    assert lib.cadd_build_workspace_bytes(C.byref(a), None) == G.ERR_NULL
    for field, bad in (("batch", 0), ("L", 65), ("K", 0), ("K", 65), ("V", 0), ("B_max", 2049), ("R", 32), ("B_max", -1)):
        b = G.BuildArgs.from_buffer_copy(a)
        setattr(b, field, bad)
        assert lib.cadd_build_workspace_bytes(C.byref(b), C.byref(out)) == G.ERR_SHAPE, field
    b = G.BuildArgs.from_buffer_copy(a); b.logits_dtype = 7
    assert lib.cadd_build_workspace_bytes(C.byref(b), C.byref(out)) == G.ERR_DTYPE
    # required pointers are checked before anything touches the device
    assert lib.cadd_build_tree(C.byref(a), None) == G.ERR_NULL
    v = G.VerifyArgs(); v.struct_size = C.sizeof(G.VerifyArgs)
    v.batch, v.L, v.R, v.V = 1, 8, 33, 1024
    assert lib.cadd_verify_tree(C.byref(v), None) == G.ERR_NULL
    v.rows_mode = 3
    assert lib.cadd_verify_tree(C.byref(v), None) == G.ERR_DTYPE
    assert G.cadd_status_string(G.ERR_WORKSPACE).startswith("workspace")
    assert G.cadd_version() == 4


def test_launch_counts_are_host_arithmetic(lib):
    """cadd_build_launches / cadd_verify_launches: one kernel per call below the small-problem sizes, two above; the flags
    that ask for the regular path or for a single kernel of it are honoured; bad shapes give the usual codes."""
    import torch
    # the five benchmark shapes: only configuration 1 is small
    assert G.cadd_round_launches(1, 8, 1024, 4, 32, 33, torch.float32) == 2
    for batch, L, K, B_max in ((32, 16, 8, 256), (128, 16, 16, 512), (64, 32, 32, 1024), (256, 16, 8, 384)):
        assert G.cadd_round_launches(batch, L, 151936, K, B_max, B_max + 1, torch.bfloat16) == 4
    a = G.BuildArgs(); a.struct_size = C.sizeof(G.BuildArgs)
    a.batch, a.L, a.V, a.K, a.B_max, a.R = 1, 8, 1024, 4, 32, 33
    a.logits_dtype = G.DTYPE_FP32
    assert lib.cadd_build_launches(C.byref(a)) == 1
    a.flags = G.FLAG_REGULAR_PATH
    assert lib.cadd_build_launches(C.byref(a)) == 2
    a.flags = G.FLAG_ONLY_TOPK
    assert lib.cadd_build_launches(C.byref(a)) == 1          # the one kernel that was asked for
    a.flags = 0
    a.V = 2049                                               # rows too long to stage: regular path
    assert lib.cadd_build_launches(C.byref(a)) == 2
    a.V, a.batch, a.L = 2048, 64, 8                          # 64 * 8 * 2048 * 4 B = 4 MiB of draft logits: regular path
    assert lib.cadd_build_launches(C.byref(a)) == 2
    a.batch = 0
    assert lib.cadd_build_launches(C.byref(a)) == G.ERR_SHAPE
    assert lib.cadd_build_launches(None) == G.ERR_NULL
    v = G.VerifyArgs(); v.struct_size = C.sizeof(G.VerifyArgs)
    v.batch, v.L, v.R, v.V = 1, 8, 33, 1024
    v.logits_dtype = G.DTYPE_FP32
    assert lib.cadd_verify_launches(C.byref(v)) == 1
    v.flags = G.VERIFY_REGULAR_PATH
    assert lib.cadd_verify_launches(C.byref(v)) == 2
    v.flags = 0
    v.V = 8193
    assert lib.cadd_verify_launches(C.byref(v)) == 2
    assert lib.cadd_verify_launches(None) == G.ERR_NULL


def test_binding_refuses_cpu_tensors():
    import torch
    with pytest.raises(ValueError):
        G.cadd_build_tree(torch.zeros(1, 2, 8), 2, 4, cost_coef=torch.ones(1, 4, dtype=torch.float64))
    with pytest.raises(ValueError):
        G.cadd_verify_tree(torch.zeros(1, 5, 8), 2, torch.zeros(1, dtype=torch.int32),
                           torch.zeros(1, 5, dtype=torch.int32), torch.zeros(1, 5, dtype=torch.int32))
