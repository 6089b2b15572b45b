"""The C ABI library builds, loads and exports every symbol include/ftc.h declares; host-only calls work
without a GPU."""
import ctypes
import os
import re

from paper_2602_22445_b200 import binding as B
from paper_2602_22445_b200 import build as cuda_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "ftc.h")).read()
    return re.findall(r"FTC_API\s+[\w\s\*]+?\b(ftc_\w+)\s*\(", text)


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(cuda_build.build())
    names = declared_symbols()
    assert len(names) >= 12 and len(set(names)) == len(names)
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(names) == sorted(B.EXPORTS)        # the binding covers the same names


def test_host_only_calls():
    assert B.ftc_version() == 0x00010000
    d = B.make_desc(65536, 8, 4, B.FTC_U64, "sum")
    s = B.ftc_schedule_info(d)
    assert (s["q"], s["r"], s["H"], s["rounds_reduce"], s["rounds_attempt"]) == (7281, 6, 13, 21, 42)
    assert (s["msgs_upcorrection"], s["msgs_tree"]) == (524274, 65535)
    assert B.ftc_kernel_name(d) == "staged" and B.ftc_workspace_bytes(d, 100) == 0
    assert B.ftc_kernel_name(B.make_desc(8, 1, 1, B.FTC_I32, "sum")) == "generic"
    assert B.ftc_workspace_bytes(B.make_desc(8, 1, 1, B.FTC_I32, "sum"), 9) == 9 * 4 * 4
    assert B.ftc_kernel_name(B.make_desc(4096, 4, 32, B.FTC_I32, "max", flags=B.FTC_KERNEL_DIRECT)) == "tiled"
    assert B.ftc_kernel_name(B.make_desc(2, 1, 1, B.FTC_I32, "sum")) == "invalid"
    # other subtree shapes: depth of the deepest node of an a-ary heap; heaps run on the level kernel where the vector is a
    # power-of-two number of 16-byte chunks, binomial trees and the rest on the general kernel
    t = B.ftc_schedule_info(B.make_desc(1024, 3, 16, B.FTC_F32, "sum", flags=B.FTC_TREE_ARITY(4)))
    assert (t["H"], t["rounds_reduce"], t["rounds_attempt"]) == (5, 8, 16)       # 256 rows: levels of 1, 4, 16, 64, 171
    assert B.ftc_kernel_name(B.make_desc(4096, 4, 32, B.FTC_I32, "max", flags=B.FTC_TREE_ARITY(3))) == "levels"
    assert B.ftc_kernel_name(B.make_desc(4096, 4, 3, B.FTC_I32, "max", flags=B.FTC_TREE_ARITY(3))) == "generic"
    assert B.ftc_kernel_name(B.make_desc(4096, 4, 32, B.FTC_I32, "max", flags=B.FTC_TREE_BINOMIAL)) == "levels"
    assert B.ftc_kernel_name(B.make_desc(4096, 4, 32, B.FTC_I32, "max", flags=B.FTC_KERNEL_LEVELS)) == "levels"
    assert B.ftc_workspace_bytes(B.make_desc(4096, 4, 32, B.FTC_I32, "max", flags=B.FTC_TREE_ARITY(3)), 1000, True) == 0
    assert B.ftc_kernel_name(B.make_desc(8, 1, 1, B.FTC_I32, "sum", flags=B.FTC_TREE_ARITY(1))) == "invalid"
    # many processes with wide vectors: the shared-memory kernel asks for a workspace for its array of tile results
    wide = B.make_desc(16384, 5, 16, B.FTC_U64, "sum")
    assert B.ftc_kernel_name(wide, True) == "staged" and B.ftc_workspace_bytes(wide, 1000, True) == 148 * 4 * 511 * 128
    assert B.ftc_kernel_name(B.make_desc(65536, 4, 32, B.FTC_I32, "max"), True) == "staged"
    for code in (0, -1, -2, -3, -4, -5):
        assert B.ftc_strerror(code) and "unknown" not in B.ftc_strerror(code)
    assert "unknown" in B.ftc_strerror(-99)
    assert B.ftc_host_staging_bytes(d, 4) >= 4 * 65536 * 32
