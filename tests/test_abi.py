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


def _readme_example():
    """The indented C example of README.md (the block that starts at the shape initialiser)."""
    lines = open(os.path.join(ROOT, "README.md")).read().splitlines()
    start = next(i for i, l in enumerate(lines) if l.startswith("    locmoe_shape_t s ="))
    block = []
    for l in lines[start:]:
        if l.strip() and not l.startswith("    "):
            break
        block.append(l)
    return "\n".join(block)


def test_readme_example_compiles_against_the_header(tmp_path):
    # the README's call sequence, wrapped in a function whose parameters are the names it uses: it must compile as
    # C99 against include/locmoe.h with every warning on (a missing argument would not)
    import shutil
    import subprocess
    gcc = shutil.which("gcc")
    if not gcc:
        pytest.skip("no host compiler")
    body = _readme_example()
    assert "locmoe_capacity_route" in body and "locmoe_combine" in body
    src = tmp_path / "readme_example.c"
    src.write_text(
        '#include "locmoe.h"\n'
        "void example(int32_t T, int32_t H, int32_t E, int32_t n_nodes, int32_t dev_per_node, const void *x, const int32_t *src_dev,\n"
        "             int32_t *idx, float *gate_w, float *cos_sim, float *delta_e, float *theta_e, locmoe_capacity_t *cap,\n"
        "             int32_t *pos, int32_t *slot, uint8_t *drop, int32_t *inv, int32_t *counts, int32_t *kept,\n"
        "             int32_t *send_counts, int32_t *load, int64_t *locality, int32_t *status, void *ws, void *buf,\n"
        "             const void *y, void *out, void *stream) {\n"
        "    int32_t C_alloc = 0; size_t ws_bytes = 0;\n" + body + "\n}\n")
    subprocess.run([gcc, "-std=c99", "-Wall", "-Wextra", "-Werror", "-I", os.path.join(ROOT, "include"), "-c", str(src),
                    "-o", str(tmp_path / "readme_example.o")], check=True)


def test_host_helpers_of_the_rule_and_the_layout(B, oracle_mod):
    import numpy as np
    from paper_2401_13920_b200 import workloads as W
    # the conventional term against the oracle's integer rule on the five configurations (its minimum does not bind
    # at delta = 0) and the three multipliers
    for w in W.CONFIGS.values():
        for cf in (1.0, 1.25, 2.0):
            idx = np.arange(w.T, dtype=np.int32) % w.E
            ref = oracle_mod.capacity(idx, np.zeros(w.T), w.E, w.H, w.D, min_mult=cf, capacity_factor=cf, delta_override=0.0)
            assert B.conventional_capacity(w.T, w.D, w.E, cf) == ref.C_local
    assert B.conventional_capacity(5, 4, 8, 1.0) == 1 and B.conventional_capacity(100, 2, 2, 0.0) == 1
    sh, rule, out = B.make_shape(100, 64, 8, 2, 2, B.F32), B.CapacityRule(1.0, 1.0, -1.0, 0, 1000), C.c_int32()
    assert B._lib.locmoe_conventional_capacity(C.byref(sh), C.byref(rule), C.byref(out)) == 0 and out.value == 32   # T_global
    rule.T_global = -1
    assert B._lib.locmoe_conventional_capacity(C.byref(sh), C.byref(rule), C.byref(out)) == -2
    # the batch-wide threshold: minimum over experts, clamped to [0, 1]; a negative minimum must not read as "measure"
    import torch
    assert B.batch_delta(torch.tensor([0.5, 0.25, 1.0])) == 0.25
    assert B.batch_delta(torch.tensor([0.5, -0.125, 1.0])) == 0.0
    assert B.batch_delta(torch.tensor([1.0, 1.0])) == 1.0
    assert B.batch_delta(torch.tensor([0.1], dtype=torch.float32)) == float(np.float32(0.1))
    d = C.c_double()
    assert B._lib.locmoe_batch_delta(None, 3, C.byref(d)) == -1
    nan = (C.c_float * 2)(0.5, float("nan"))
    assert B._lib.locmoe_batch_delta(C.cast(nan, C.c_void_p), 2, C.byref(d)) == -2
    # r(a, b) against the oracle's destination orders
    for N, Dn in ((2, 2), (1, 4), (4, 8), (3, 1)):
        r = oracle_mod.dest_order(N, Dn)              # r[a][b]
        D = N * Dn
        for a in range(D):
            for b in range(D):
                assert B.dest_order(N, Dn, a, b) == int(r[a][b])
    # device 1 of a 2 x 2 map lists itself, its node neighbour 0, then the other node's 3 and 2
    assert [B.dest_order(2, 2, 1, b) for b in (1, 0, 3, 2)] == [0, 1, 2, 3]
    assert B._lib.locmoe_dest_order(C.byref(B.make_shape(1, 1, 1, 2, 2, B.F32)), 0, 4) == -2


def test_ffn_kernel_choice_is_a_host_side_query(B, monkeypatch):
    # no launch, no device needed (the SM count falls back to a B200's 148): config 5's full size takes the wide kernel for
    # the long reduction only; small batches and forced choices behave as documented
    monkeypatch.delenv("LOCMOE_FFN", raising=False)
    sh = B.make_shape(65536, 2560, 32, 4, 8, B.BF16, B.LAYOUT_RECV)
    assert B.locmoe_ffn_kernels(sh, 64, 10240) == (0, 1)         # 2048 rows per expert
    assert B.locmoe_ffn_kernels(sh, 8, 10240) == (0, 1)          # 256 rows per expert: 320 wide tiles, the last 24 as halves
    assert B.locmoe_ffn_kernels(sh, 4, 10240) == (0, 0)          # 128 rows per expert: half of every 256-row tile would be empty
    assert B.locmoe_ffn_kernels(sh, 32, 10240) == (0, 1)         # 1024 rows per expert
    assert B.locmoe_ffn_kernels(sh, 64, 4096) == (0, 0)          # no reduction long enough
    assert B.locmoe_ffn_kernels(sh, 64, 5120) == (0, 1)          # 5120 is, without a GeLU in the epilogue
    sh3 = B.make_shape(65536, 2560, 32, 4, 8, B.BF16, B.LAYOUT_RECV)
    assert B.locmoe_ffn_kernels(sh3, 3, 10240) == (0, 0)         # 96 rows per expert: a 256-row tile would be mostly empty
    monkeypatch.setenv("LOCMOE_FFN", "w")
    assert B.locmoe_ffn_kernels(sh, 8, 10240) == (1, 1)
    monkeypatch.setenv("LOCMOE_FFN", "w1")
    assert B.locmoe_ffn_kernels(sh, 8, 10240) == (1, 0)
    monkeypatch.setenv("LOCMOE_FFN", "1")
    assert B.locmoe_ffn_kernels(sh, 64, 10240) == (0, 0)
    monkeypatch.setenv("LOCMOE_FFN", "2s")
    assert B.locmoe_ffn_kernels(sh, 64, 10240) == (3, 3)
    import ctypes as C
    assert B._lib.locmoe_ffn_kernels(C.byref(sh), 64, 10244, C.byref((C.c_int32 * 2)())) == -2
    assert B._lib.locmoe_ffn_kernels(C.byref(sh), 64, 10240, None) == -1
