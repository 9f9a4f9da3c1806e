"""GPU parity of the expert FFN (tcgen05 grouped GEMMs) and of the whole-layer call against the CPU oracle.

Tolerance, from the arithmetic: the kernels take bf16 inputs, accumulate in fp32 and round the intermediate
g = GeLU(W_in x) to bf16 (8 significant bits: relative error at most 2^-8 per element, independent signs), then accumulate
y = sum_f W_out[i][f] g[f] in fp32 and round y to bf16.  With s_i = sqrt(sum_f (W_out[i][f] g[f])^2) (returned by
the oracle) the deviation from the fp64 oracle is bounded, with wide margin, by
    6 * 2^-8 / sqrt(3) * s_i   (intermediate rounding: six standard deviations of a uniform error)
  + 2^-8 * |y_i|               (final bf16 rounding, half an ulp is at most |y| / 256)
  + 1e-6 * sum-scale           (fp32 accumulation).
"""
import os

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

# The two-SM kernel is opt-in in the library (LOCMOE_FFN=2) and therefore in the tests as well: its launches failed
# under multi-metric profiler captures for a reason that has not been found, so a default test run leaves it alone.
# LOCMOE_TEST_FFN2=1 runs its cases.
two_sm = pytest.mark.skipif(os.environ.get("LOCMOE_TEST_FFN2") != "1", reason="two-SM FFN kernel is opt-in (LOCMOE_TEST_FFN2=1)")


@pytest.fixture(scope="module")
def P():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    import oracle
    oracle.build()
    from tests import parity
    return parity


def _tol(y, spread, out_is_bf16):
    t = 6.0 * 2.0 ** -8 / np.sqrt(3.0) * spread + 1e-5 * spread + 1e-7
    if out_is_bf16:
        t = t + 2.0 ** -8 * np.abs(y)
    return t


def _check_rows(P, buf, w_in, w_out, y, E, M, rows, y_is_bf16=True):
    W = P.W
    for r in rows:
        e = r // M
        want, spread = P.oracle.ffn_rows(W.host_bits(buf[r:r + 1]), W.host_bits(w_in[e]), W.host_bits(w_out[e]))
        got = y[r].double().cpu().numpy()
        err = np.abs(got - want[0])
        assert (err <= _tol(want[0], spread[0], y_is_bf16)).all(), "row %d: max err %.4g" % (r, err.max())


@pytest.mark.parametrize("E,N,Dn,C,H,F,ydt", [
    (2, 1, 2, 32, 64, 256, torch.bfloat16),      # M = 64: less than one tile
    (4, 2, 2, 70, 264, 520, torch.bfloat16),     # M = 280, K and N with ragged tails
    (4, 2, 2, 70, 264, 520, torch.float32),
    (8, 1, 8, 40, 512, 1024, torch.bfloat16),    # M = 320, several k-blocks and n-tiles
    (2, 1, 2, 300, 320, 512, torch.bfloat16),    # M = 600: three 256-row tiles, the last one with an empty lower half
    (4, 1, 2, 256, 64, 5120, torch.bfloat16),    # first GEMM: 160 tiles of 256 x 256 -- on 148 SMs the wide kernel splits the last 12 into halves
    (4, 1, 2, 300, 64, 3328, torch.bfloat16),    # M = 600 and 156 wide tiles: split halves that lie wholly beyond an expert's rows
])
@pytest.mark.parametrize("kernel", ["one_sm", "wide", pytest.param("two_sm_single_acc", marks=two_sm), pytest.param("two_sm", marks=two_sm)])
def test_expert_ffn_small_shapes_all_rows(P, monkeypatch, kernel, E, N, Dn, C, H, F, ydt):
    # LOCMOE_FFN=2 selects the two-SM kernel (cluster of two CTAs, tcgen05 cta_group::2), 2s its one-accumulator form
    # and w the wide kernel (256 x 256 tiles, one CTA each) for both GEMMs
    monkeypatch.setenv("LOCMOE_FFN", {"one_sm": "1", "wide": "w", "two_sm_single_acc": "2s", "two_sm": "2"}[kernel])
    B = P.B
    dev = torch.device("cuda:0")
    D = N * Dn
    rows, M = D * E * C, D * C
    g = torch.Generator(device=dev).manual_seed(5)
    buf = torch.randn(rows, H, generator=g, device=dev).to(torch.bfloat16)
    buf[3] = 0                                                    # an empty slot stays empty
    w_in = (torch.randn(E, F, H, generator=g, device=dev) * 0.08).to(torch.bfloat16)
    w_out = (torch.randn(E, H, F, generator=g, device=dev) * 0.08).to(torch.bfloat16)
    sh = B.make_shape(rows, H, E, N, Dn, torch.bfloat16, B.LAYOUT_RECV)
    h1 = torch.empty(rows, F, dtype=torch.bfloat16, device=dev)
    y = torch.full((rows, H), 7.0, dtype=ydt, device=dev)
    B.locmoe_expert_ffn(sh, C, F, buf, w_in, w_out, h1, y)
    torch.cuda.synchronize()
    assert B.locmoe_device_flags() == 0
    assert not y[3].any().item()
    _check_rows(P, buf, w_in, w_out, y, E, M, range(rows), ydt == torch.bfloat16)


def _random_shapes(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    for _ in range(n):
        Dn = int(rng.choice([1, 2, 4]))
        E = Dn * int(rng.choice([1, 2, 3]))       # the experts divide evenly over the devices
        C = int(rng.integers(1, 160))            # M = Dn * C rows per expert: from 1 to several tiles, any remainder
        H = 8 * int(rng.integers(1, 60))          # rows of 16 bytes and more, reductions that end inside a k-block
        F = 8 * int(rng.integers(1, 90))
        out.append((E, Dn, C, H, F))
    return out


@pytest.mark.parametrize("E,Dn,C,H,F", _random_shapes(8, 20240113))
@pytest.mark.parametrize("kernel", ["one_sm", "wide"])
def test_expert_ffn_random_ragged_shapes(P, monkeypatch, kernel, E, Dn, C, H, F):
    # seeded random shapes, every row checked: tiles cut by the rows of an expert, by N and by K in either kernel
    monkeypatch.setenv("LOCMOE_FFN", {"one_sm": "1", "wide": "w"}[kernel])
    B = P.B
    dev = torch.device("cuda:0")
    rows, M = Dn * E * C, Dn * C
    g = torch.Generator(device=dev).manual_seed(E * 1000 + C)
    buf = torch.randn(rows, H, generator=g, device=dev).to(torch.bfloat16)
    w_in = (torch.randn(E, F, H, generator=g, device=dev) * 0.1).to(torch.bfloat16)
    w_out = (torch.randn(E, H, F, generator=g, device=dev) * 0.1).to(torch.bfloat16)
    sh = B.make_shape(rows, H, E, 1, Dn, torch.bfloat16, B.LAYOUT_RECV)
    h1 = torch.full((rows, F), 3.0, dtype=torch.bfloat16, device=dev)
    y = torch.full((rows, H), 7.0, dtype=torch.bfloat16, device=dev)
    B.locmoe_expert_ffn(sh, C, F, buf, w_in, w_out, h1, y)
    torch.cuda.synchronize()
    assert B.locmoe_device_flags() == 0
    _check_rows(P, buf, w_in, w_out, y, E, M, range(rows))


def test_expert_ffn_rejects_send_layout_and_bad_sizes(P):
    B = P.B
    import ctypes as C
    one = C.c_void_p(256)
    sh = B.make_shape(64, 64, 2, 1, 2, B.BF16, B.LAYOUT_SEND)
    assert B._lib.locmoe_expert_ffn(C.byref(sh), 4, 64, one, one, one, one, one, B.BF16, None) == -3
    sh = B.make_shape(64, 64, 2, 1, 2, B.BF16, B.LAYOUT_RECV)
    assert B._lib.locmoe_expert_ffn(C.byref(sh), 4, 60, one, one, one, one, one, B.BF16, None) == -2
    assert B._lib.locmoe_expert_ffn(C.byref(sh), 4, 64, C.c_void_p(8), one, one, one, one, B.BF16, None) == -4


@pytest.mark.parametrize("kernel", ["one_sm", "wide", pytest.param("two_sm", marks=two_sm)])
def test_full_layer_config5_scaled(P, monkeypatch, kernel):
    # config 5: router + dispatch (RECV layout), expert FFN with random-init weights, combine; one C-ABI call
    monkeypatch.setenv("LOCMOE_FFN", {"one_sm": "1", "wide": "w", "two_sm": "2"}[kernel])
    W, B = P.W, P.B
    dev = torch.device("cuda:0")
    w = W.CONFIGS[5].scaled(8192)
    F = 10240
    x = W.make_tokens(w, dev)
    src = W.make_src(w, dev)
    w_in, w_out = W.make_expert_weights(w, F, dev)
    sh = B.make_shape(w.T, w.H, w.E, w.n_nodes, w.dev_per_node, x.dtype, B.LAYOUT_RECV)
    rule = B.CapacityRule(1.0, 1.0, -1.0, 0, 0)
    Ca = B.conventional_capacity(w.T, sh.D, w.E, 1.0)
    st = B.make_router(sh, Ca, rule, dev)
    h1 = torch.empty(st.rows, F, dtype=torch.bfloat16, device=dev)
    y = torch.empty(st.rows, w.H, dtype=torch.bfloat16, device=dev)
    B.locmoe_moe_layer(sh, x, src, None, rule, Ca, F, w_in, w_out, B.layer_buffers(st, h1, y), st.out)
    torch.cuda.synchronize()
    assert B.locmoe_device_flags() == 0
    # router stages against the oracle
    gi = P.check_gate(x, sh, st)
    cap, ref_cap = P.check_capacity(sh, st, rule, gi)
    rr = P.check_route(sh, st, src, cap, gi, ref_cap)
    P.check_dispatch_full(x, sh, st, rr)
    # expert outputs of sampled occupied and empty rows
    rng = np.random.default_rng(3)
    occ = np.nonzero(rr.inv >= 0)[0]
    emp = np.nonzero(rr.inv < 0)[0]
    rows = np.concatenate([rng.choice(occ, 12, replace=False), emp[:2]])
    _check_rows(P, st.buf, w_in, w_out, y, w.E, st.rows // w.E, [int(r) for r in rows])
    # combine of the FFN output
    toks = np.unique(np.concatenate([rng.integers(0, w.T, 256), np.nonzero(rr.drop)[0][:16]]))
    P.check_combine_sampled(y, sh, st, rr, gi, toks)


def test_full_layer_config5_full_size(P):
    # config 5 at its full size (T = 65536, 2048 rows per expert, F = 10240: 20480 tiles per GEMM) through the one
    # layer call, default (one-SM) kernel: router stages against the oracle, sampled expert-output rows (occupied and
    # empty) and sampled combined tokens against the fp64 oracle
    W, B = P.W, P.B
    dev = torch.device("cuda:0")
    w = W.CONFIGS[5]
    F = 10240
    x = W.make_tokens(w, dev)
    src = W.make_src(w, dev)
    w_in, w_out = W.make_expert_weights(w, F, dev)
    sh = B.make_shape(w.T, w.H, w.E, w.n_nodes, w.dev_per_node, x.dtype, B.LAYOUT_RECV)
    rule = B.CapacityRule(1.0, 1.0, -1.0, 0, 0)
    Ca = B.conventional_capacity(w.T, sh.D, w.E, 1.0)
    assert Ca == 64
    st = B.make_router(sh, Ca, rule, dev)
    h1 = torch.empty(st.rows, F, dtype=torch.bfloat16, device=dev)
    y = torch.full((st.rows, w.H), 7.0, dtype=torch.bfloat16, device=dev)
    B.locmoe_moe_layer(sh, x, src, None, rule, Ca, F, w_in, w_out, B.layer_buffers(st, h1, y), st.out)
    torch.cuda.synchronize()
    assert B.locmoe_device_flags() == 0
    gi = P.check_gate(x, sh, st)
    assert gi["n_differ"] == 0
    cap, ref_cap = P.check_capacity(sh, st, rule, gi)
    assert (ref_cap.C_local, ref_cap.C_expert) == (cap.C_local, cap.C_expert) == (64, 2048)
    rr = P.check_route(sh, st, src, cap, gi, ref_cap)
    rng = np.random.default_rng(11)
    P.check_dispatch_sampled(x, sh, st, rr, np.unique(rng.integers(0, st.rows, 1024)))
    occ = np.nonzero(rr.inv >= 0)[0]
    emp = np.nonzero(rr.inv < 0)[0]
    assert len(emp) >= 2
    M = st.rows // w.E
    # rows from the first and last tile of an expert, the first and last expert, and random ones in between
    picks = [occ[0], occ[-1], occ[occ >= 17 * M][0], occ[occ < 18 * M][-1]]
    picks += list(rng.choice(occ, 14, replace=False)) + [emp[0], emp[-1]]
    _check_rows(P, st.buf, w_in, w_out, y, w.E, M, [int(r) for r in picks])
    assert not y[int(emp[0])].any().item() and not y[int(emp[-1])].any().item()
    toks = np.unique(np.concatenate([rng.integers(0, w.T, 256), [0, w.T - 1], np.nonzero(rr.drop)[0][:16]]))
    P.check_combine_sampled(y, sh, st, rr, gi, toks)
    del h1, y, w_in, w_out, st
    torch.cuda.empty_cache()


def test_layer_call_with_identity_experts_equals_the_five_calls(P):
    W, B = P.W, P.B
    dev = torch.device("cuda:0")
    w = W.CONFIGS[2].scaled(5000)
    x = W.make_tokens(w, dev)
    src = W.make_src(w, dev)
    sh = B.make_shape(w.T, w.H, w.E, w.n_nodes, w.dev_per_node, x.dtype)
    rule = B.CapacityRule(1.25, 1.25, -1.0, 0, 0)
    Ca = B.conventional_capacity(w.T, sh.D, w.E, 1.25)
    a = B.make_router(sh, Ca, rule, dev)
    b = B.make_router(sh, Ca, rule, dev)
    B.router_forward(a, x, src)
    B.locmoe_moe_layer(sh, x, src, None, rule, Ca, 0, None, None, B.layer_buffers(b), b.out)
    torch.cuda.synchronize()
    for name in ("idx", "gate_w", "cos_sim", "pos", "slot", "drop", "inv", "counts", "kept", "send_counts", "load",
                 "locality", "status"):
        assert torch.equal(getattr(a, name), getattr(b, name)), name
    assert torch.equal(a.buf.view(torch.int16), b.buf.view(torch.int16))
    assert torch.equal(a.out.view(torch.int16), b.out.view(torch.int16))
