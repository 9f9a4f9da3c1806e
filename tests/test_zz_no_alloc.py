"""The no-allocation capacity entry point against the ordinary one.

Some hosts of this library cannot allocate device memory at all -- a plug-in
inside a serving process that has already reserved the whole HBM, or a C caller
that is handed only an operator's input and output buffers -- so they cannot
supply the workspace `locmoe_capacity` asks for.  `locmoe_capacity_noalloc`
keeps that scratch in a fixed array inside the library instead.  This test
calls it through the C ABI twice in a row, on different problems (the second
call finds the first call's leftovers in the shared array), and requires the
very same outputs as `locmoe_capacity` gives with a caller workspace -- and,
so that the comparison does not rest on CUDA agreeing with CUDA, the values the
CPU oracle computes from the same index and cosine arrays.  It also checks
that the call really allocates nothing (free device memory and torch's
allocator statistics are unchanged across it), and runs the same comparison in
a child process that forces the multi-kernel path (memset + grid-wide minimum
+ finish kernel) through the built-in array.

Collected last on purpose (file name), so that a run stopping at the first
failure has already run every other test; it also passes on its own.
"""
import ctypes as C
import math
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _problem(B, W, cfg, T, rule, dev):
    w = W.CONFIGS[cfg].scaled(T)
    x = W.make_tokens(w, dev)
    sh = B.make_shape(w.T, w.H, w.E, w.n_nodes, w.dev_per_node, x.dtype)
    idx = torch.empty(w.T, dtype=torch.int32, device=dev)
    gw = torch.empty(w.T, device=dev)
    cs = torch.empty(w.T, device=dev)
    B.locmoe_gate(sh, x, None, idx, gw, cs)
    return sh, idx, cs


def _run(B, sh, idx, cs, rule, dev, noalloc):
    de = torch.full((sh.E,), -7.0, device=dev)
    te = torch.full((sh.E,), -7.0, device=dev)
    cap = torch.zeros(B.CAPACITY_BYTES, dtype=torch.uint8, device=dev)
    if noalloc:
        B.locmoe_capacity_noalloc(sh, idx, cs, rule, de, te, cap)
    else:
        ws = torch.empty(B.locmoe_workspace_bytes(sh, 1), dtype=torch.uint8, device=dev)
        B.locmoe_capacity(sh, idx, cs, rule, de, te, cap, ws)
    rec = B.locmoe_capacity_read(cap)
    return de, te, rec


def _same(a, b):
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
    ra, rb = a[2], b[2]
    for f in ("delta", "p_delta", "ec_min", "C_expert", "C_local", "n_empty_experts", "flags"):
        assert getattr(ra, f) == getattr(rb, f), f


def _against_oracle(got, sh, idx, cs, rule):
    """delta_e, the record and the integer capacities against the CPU oracle on the same (idx, cos) arrays."""
    import oracle
    oracle.build()
    de, te, rec = got
    ref = oracle.capacity(idx.cpu().numpy(), cs.double().cpu().numpy(), sh.E, sh.H, sh.D, rule.min_mult,
                          rule.capacity_factor, rule.delta_override, rule.bound_form)
    assert np.array_equal(de.cpu().numpy(), ref.delta_e.astype(np.float32))
    assert np.allclose(te.cpu().numpy(), np.arccos(np.clip(ref.delta_e, -1, 1)), rtol=1e-6, atol=1e-6)
    assert rec.delta == ref.delta and rec.n_empty_experts == ref.n_empty_experts
    assert math.isclose(rec.p_delta, ref.p_delta, rel_tol=1e-8, abs_tol=1e-300)
    assert math.isclose(rec.ec_min, ref.ec_min, rel_tol=1e-8)
    assert (rec.C_expert, rec.C_local) == (ref.C_expert, ref.C_local)


def _twice_in_a_row(check_memory):
    from paper_2401_13920_b200 import binding as B
    from paper_2401_13920_b200 import workloads as W
    dev = torch.device("cuda:0")
    rule_a = B.CapacityRule(1.0, 1.0, -1.0, B.BOUND_BETA, 0)
    rule_b = B.CapacityRule(2.0, 1.25, -1.0, B.BOUND_ERFC, 0)
    prob_a = _problem(B, W, 4, 9001, rule_a, dev)     # 256 experts
    prob_b = _problem(B, W, 1, 4096, rule_b, dev)     # 8 experts: most of the shared array keeps call 1's data
    want_a = _run(B, *prob_a, rule_a, dev, noalloc=False)
    want_b = _run(B, *prob_b, rule_b, dev, noalloc=False)
    got_a = _run(B, *prob_a, rule_a, dev, noalloc=True)      # first call: also looks up the array's address
    got_b = _run(B, *prob_b, rule_b, dev, noalloc=True)      # second call, right after, on a different problem
    _same(got_a, want_a)
    _same(got_b, want_b)
    _against_oracle(got_a, *prob_a, rule_a)
    _against_oracle(got_b, *prob_b, rule_b)
    if check_memory:
        # a further call with every output already in place: neither the driver's free memory nor torch's
        # allocator may move across it
        sh, idx, cs = prob_b
        de = torch.empty(sh.E, device=dev); te = torch.empty(sh.E, device=dev)
        cap = torch.zeros(B.CAPACITY_BYTES, dtype=torch.uint8, device=dev)
        torch.cuda.synchronize()
        free0, _ = torch.cuda.mem_get_info(dev)
        stats0 = (torch.cuda.memory_allocated(dev), torch.cuda.memory_reserved(dev))
        B.locmoe_capacity_noalloc(sh, idx, cs, rule_b, de, te, cap)
        torch.cuda.synchronize()
        free1, _ = torch.cuda.mem_get_info(dev)
        assert free1 == free0 and (torch.cuda.memory_allocated(dev), torch.cuda.memory_reserved(dev)) == stats0
        assert torch.equal(de, want_b[0])
    assert want_a[2].C_local == 1 and want_b[2].C_local == 80
    # and once more on the first problem: the array now holds call 2's leftovers
    _same(_run(B, *prob_a, rule_a, dev, noalloc=True), want_a)
    assert B.locmoe_device_flags() == 0


def test_noalloc_capacity_matches_the_workspace_entry_point_twice_in_a_row():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    _twice_in_a_row(check_memory=True)


def test_noalloc_capacity_multi_kernel_path_through_the_builtin_array():
    # LOCMOE_PATH=grid (read at call time, but kept out of this process's environment) forces memset + grid-wide
    # minimum + finish kernel, the path large batches take, through the built-in array
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    code = "from tests import test_zz_no_alloc as t; t._twice_in_a_row(False); print('ok')"
    r = subprocess.run([sys.executable, "-c", code], cwd=root, env=dict(os.environ, LOCMOE_PATH="grid"),
                       capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and r.stdout.strip().endswith("ok"), r.stderr[-2000:]


def test_noalloc_capacity_rejects_a_negative_global_token_count():
    from paper_2401_13920_b200 import binding as B
    sh = B.make_shape(64, 64, 8, 1, 2, B.BF16)
    rule = B.CapacityRule(1.0, 1.0, -1.0, 0, -5)
    one = C.c_void_p(256)
    assert B._lib.locmoe_capacity_noalloc(C.byref(sh), one, one, C.byref(rule), one, one, one, None) == -2


def test_noalloc_capacity_rejects_more_experts_than_its_scratch_holds():
    from paper_2401_13920_b200 import binding as B
    sh = B.make_shape(64, 16384, 16384, 1, 1, B.BF16)        # 16384 experts > 8192
    rule = B.CapacityRule(1.0, 1.0, -1.0, 0, 0)
    one = C.c_void_p(256)                                      # never dereferenced: the size check comes first
    rc = B._lib.locmoe_capacity_noalloc(C.byref(sh), one, one, C.byref(rule), one, one, one, None)
    assert rc == -7 and "scratch" in B.status_string(rc)
