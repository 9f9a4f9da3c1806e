"""The C-ABI library loads, exports every function the header declares, and
rejects bad arguments on the host (no GPU needed: nothing is launched)."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_2401_13920_b200 import binding
    return binding


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "locmoe.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(locmoe_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(B):
    names = _declared_functions()
    assert set(B.EXPORTS) <= set(names) and len(names) >= 8
    lib = C.CDLL(B.library_path())
    for n in names:
        assert hasattr(lib, n), n


def test_struct_layouts_match_the_header(B):
    assert C.sizeof(B.Shape) == 28
    assert C.sizeof(B.CapacityRule) == 32
    assert C.sizeof(B.Capacity) == 40


def test_status_strings(B):
    assert B.status_string(0) == "ok"
    for code in range(-6, 0):
        assert B.status_string(code) not in ("ok", "unknown error")
    assert B.status_string(-99) == "unknown error"


def test_workspace_query_and_shape_validation(B):
    sh = B.make_shape(65536, 5120, 64, 8, 8, B.BF16)
    n = B.locmoe_workspace_bytes(sh, 16)
    assert n % 256 == 0 and n >= 4 * 65536 * 4
    small = B.locmoe_workspace_bytes(B.make_shape(4096, 1024, 8, 2, 4, B.F32), 64)
    assert 0 < small < n
    lib = B._lib
    out = C.c_size_t()
    for bad in [B.make_shape(0, 1024, 8, 2, 4, B.F32),          # no tokens
                B.make_shape(16, 1000, 7, 1, 1, B.F32),          # H % E != 0
                B.make_shape(16, 1024, 8, 3, 1, B.F32),          # E % D != 0
                B.make_shape(16, 1024, 8, 4, 4, B.F32)]:         # more devices than experts
        assert lib.locmoe_workspace_bytes(C.byref(bad), 4, C.byref(out)) == -2
    assert lib.locmoe_workspace_bytes(C.byref(B.make_shape(16, 1024, 8, 2, 4, 7)), 4, C.byref(out)) == -3
    assert lib.locmoe_workspace_bytes(C.byref(sh), 0, C.byref(out)) == -2
    assert lib.locmoe_workspace_bytes(C.byref(sh), 2 ** 30, C.byref(out)) == -2   # rows overflow int32
    assert lib.locmoe_workspace_bytes(None, 4, C.byref(out)) == -1


def test_null_pointers_are_rejected_before_any_launch(B):
    lib = B._lib
    sh = B.make_shape(16, 64, 8, 2, 4, B.F32)
    assert lib.locmoe_gate(C.byref(sh), None, None, None, None, None, None, None) == -1
    assert lib.locmoe_dispatch(C.byref(sh), 4, None, None, None, None, 1, None) == -1
    assert lib.locmoe_combine(C.byref(sh), 4, None, 0, None, None, None, 0, None) == -1
    assert lib.locmoe_loc_loss(C.byref(sh), None, 0, 1.0, 1e-3, None, None, None, None, None) == -1
    assert lib.locmoe_topk_select(C.byref(sh), None, None, None, 2, None, None, None) == -1
    assert lib.locmoe_topk_fold(C.byref(sh), 4, None, None) == -1
    assert lib.locmoe_combine_topk(C.byref(sh), 4, None, 0, 2, None, None, None, None) == -1
    assert lib.locmoe_dispatch_peer(C.byref(sh), 4, None, None, None, None, 1, 0, 1, 1, None) == -1
    assert lib.locmoe_combine_peer(C.byref(sh), 4, None, 1, 0, None, None, None, None) == -1
    assert lib.locmoe_cos_hist(C.byref(sh), None, None, 0, 1, 8, -1.0, 1.0, None, None, None, None) == -1
    rule = B.CapacityRule(1.0, 1.0, -1.0, 0, 0)
    assert lib.locmoe_capacity(C.byref(sh), None, None, C.byref(rule), None, None, None, None, 0, None) == -1
    assert lib.locmoe_gate_route(C.byref(sh), None, None, None, C.byref(rule), *([None] * 6), 4, *([None] * 10), 0, None, 0, None) == -1
    assert lib.locmoe_route(C.byref(sh), None, None, None, 4, *([None] * 10), None, 0, None) == -1
    assert lib.locmoe_capacity_route(C.byref(sh), None, None, None, C.byref(rule), None, None, None, 4, *([None] * 10),
                                     0, None, 0, None) == -1


def test_header_is_plain_c_and_links_from_a_c_program(tmp_path):
    # the boundary is a C ABI: the header must compile as C99 (and C++), and a C program must link against the library
    import shutil
    import subprocess
    from paper_2401_13920_b200 import build
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    hdr = os.path.join(root, "include", "locmoe.h")
    gcc, gxx = shutil.which("gcc"), shutil.which("g++")
    if not gcc or not gxx:
        pytest.skip("no host compiler")
    subprocess.run([gcc, "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-fsyntax-only", "-x", "c", hdr], check=True)
    subprocess.run([gxx, "-std=c++17", "-Wall", "-Werror", "-fsyntax-only", "-x", "c++", hdr], check=True)
    src = tmp_path / "probe.c"
    src.write_text(
        '#include <stdio.h>\n#include "locmoe.h"\n'
        "int main(void) {\n"
        "    locmoe_shape_t s = {4096, 1024, 8, 2, 4, LOCMOE_F32, LOCMOE_LAYOUT_SEND};\n"
        "    size_t bytes = 0;\n"
        "    int rc = locmoe_workspace_bytes(&s, 64, &bytes);\n"
        '    printf("%d %zu %s\\n", rc, bytes, locmoe_status_string(LOCMOE_ERR_SHAPE));\n'
        "    s.H = 1023;\n"
        "    return locmoe_workspace_bytes(&s, 64, &bytes) == LOCMOE_ERR_SHAPE && rc == LOCMOE_OK && bytes > 0 ? 0 : 1;\n"
        "}\n")
    lib = build.build()
    exe = tmp_path / "probe"
    subprocess.run([gcc, "-std=c99", "-I", os.path.join(root, "include"), str(src), "-o", str(exe), lib,
                    "-Wl,-rpath," + os.path.dirname(lib)], check=True)
    r = subprocess.run([str(exe)], capture_output=True, text=True)
    assert r.returncode == 0, r.stdout + r.stderr
    assert r.stdout.split()[0] == "0" and "invalid shape" in r.stdout
