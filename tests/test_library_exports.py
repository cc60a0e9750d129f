"""The C-ABI library builds, loads and exports every function include/qsim.h declares (no GPU needed)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "qsim.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(qsim_[a-z_]+)\s*\(", text)))


def test_header_declares_the_boundary_calls():
    names = declared_functions()
    for n in ("qsim_create", "qsim_run", "qsim_stats", "qsim_bind", "qsim_workspace_bytes", "qsim_destroy"):
        assert n in names


def test_library_builds_and_exports_every_declared_symbol():
    from paper_2602_02987_b200 import build_library
    from paper_2602_02987_b200.binding import EXPORTS
    lib = ctypes.CDLL(build_library())
    names = declared_functions()
    for n in names:
        assert hasattr(lib, n), f"{n} declared in qsim.h but not exported"
    assert set(EXPORTS) == set(names)


def test_binding_struct_layouts_match_the_header_sizes():
    from paper_2602_02987_b200 import binding as b
    # sizes implied by the header's field lists (natural alignment)
    assert ctypes.sizeof(b.qsim_config) == 14 * 4 + 2 * 8 + 8
    assert ctypes.sizeof(b.qsim_class) == 24
    assert ctypes.sizeof(b.qsim_targets) == 8 + 6 * 8 * 8
    assert ctypes.sizeof(b.qsim_class_stats) == 14 * 8 + 6 * 4 + 7 * 8
    assert ctypes.sizeof(b.qsim_rep_stats) == 8 * ctypes.sizeof(b.qsim_class_stats) + 6 * 8


def test_oracle_and_cuda_path_share_no_code():
    # neither side imports or includes the other
    for root, _, files in os.walk(os.path.join(ROOT, "paper_2602_02987_b200")):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(root, f)).read()
                assert "oracle" not in src.lower(), f
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c", ".h")):
            src = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2602_02987_b200" not in src and "qsim.h" not in src, f
