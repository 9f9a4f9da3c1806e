"""The no-allocation capacity entry point against the ordinary one.

Some hosts of this library cannot allocate device memory at all -- a plug-in
inside a serving process that has already reserved the whole HBM, or a C caller
that is handed only an operator's input and output buffers -- so they cannot
supply the workspace `locmoe_capacity` asks for.  `locmoe_capacity_noalloc`
keeps that scratch in a fixed array inside the library instead.  This test
calls it through the C ABI twice in a row, on different problems (the second
call finds the first call's leftovers in the shared array), and requires the
very same outputs as `locmoe_capacity` gives with a caller workspace.

Collected last on purpose (file name), so that a run stopping at the first
failure has already run every other test; it also passes on its own.
"""
import ctypes as C

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


def test_noalloc_capacity_matches_the_workspace_entry_point_twice_in_a_row():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
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
    assert want_a[2].C_local == 1 and want_b[2].C_local == 80
    # and once more on the first problem: the array now holds call 2's leftovers
    _same(_run(B, *prob_a, rule_a, dev, noalloc=True), want_a)
    assert B.locmoe_device_flags() == 0


def test_noalloc_capacity_rejects_more_experts_than_its_scratch_holds():
    from paper_2401_13920_b200 import binding as B
    sh = B.make_shape(64, 16384, 16384, 1, 1, B.BF16)        # 16384 experts > 8192
    rule = B.CapacityRule(1.0, 1.0, -1.0, 0, 0)
    one = C.c_void_p(256)                                      # never dereferenced: the size check comes first
    rc = B._lib.locmoe_capacity_noalloc(C.byref(sh), one, one, C.byref(rule), one, one, one, None)
    assert rc == -7 and "scratch" in B.status_string(rc)
