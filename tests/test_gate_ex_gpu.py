"""GPU parity of the gate's extras (locmoe_gate_ex): the per-source-device bias table against the oracle, and the
column sums of the probabilities formed inside the gate kernel against the oracle's auxiliary loss."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def P():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    import oracle
    oracle.build()
    from tests import parity
    return parity


SHAPES = [
    dict(T=6000, H=5120, E=64, n_nodes=8, dev_per_node=8, dtype="bf16"),    # specialised kernel (config 2's shape)
    dict(T=7001, H=2560, E=32, n_nodes=4, dev_per_node=8, dtype="bf16"),    # specialised kernel, five vectors per chunk
    dict(T=5003, H=5120, E=256, n_nodes=32, dev_per_node=8, dtype="bf16"),  # specialised kernel, eight groups per lane
    dict(T=4096, H=1024, E=8, n_nodes=2, dev_per_node=4, dtype="f32"),      # general vector kernel, several lanes per group
    dict(T=777, H=60, E=4, n_nodes=1, dev_per_node=4, dtype="f32"),         # general vector kernel, ragged chunks
    dict(T=777, H=36, E=4, n_nodes=2, dev_per_node=2, dtype="bf16"),        # scalar kernel
    dict(T=3, H=64, E=4, n_nodes=1, dev_per_node=2, dtype="bf16"),          # fewer rows than warps in a CTA
]


def _setup(P, kw):
    W, B = P.W, P.B
    dev = torch.device("cuda:0")
    w = W.Workload(name="gate_ex", config=6, tokens="normal", src="uniform", **kw)
    x, src = W.make_tokens(w, dev), W.make_src(w, dev)
    sh = B.make_shape(w.T, w.H, w.E, w.n_nodes, w.dev_per_node, x.dtype)
    idx = torch.empty(w.T, dtype=torch.int32, device=dev)
    gw = torch.empty(w.T, device=dev)
    cs = torch.empty(w.T, device=dev)
    return w, dev, x, src, sh, idx, gw, cs


@pytest.mark.parametrize("kw", SHAPES)
def test_per_source_bias_table(P, kw):
    W, B, oracle = P.W, P.B, P.oracle
    w, dev, x, src, sh, idx, gw, cs = _setup(P, kw)
    D = sh.D
    rng = np.random.default_rng(17)
    table = rng.uniform(-0.08, 0.08, (D, w.E)).astype(np.float32)
    src = src.clone()
    if w.T > 10:
        src[5] = D + 3                                           # an impossible source: no bias for that token
    probs = torch.empty(w.T, w.E, device=dev)
    B.locmoe_gate_ex(sh, x, idx, gw, cs, eps=torch.as_tensor(table, device=dev), src_dev=src, probs=probs)
    torch.cuda.synchronize()
    ref = oracle.gate_per_source(W.host_bits(x), sh.x_dtype, w.E, table, src.cpu().numpy(), want_probs=True)
    differ = idx.cpu().numpy() != ref.idx
    assert (ref.gap[differ] < P.GAP_EXCUSE).all(), "expert index differs on a token that is no near-tie"
    same = ~differ
    assert (np.abs(gw.cpu().numpy()[same] - ref.R[same]) <= P.GATE_RTOL * ref.R[same]).all()
    assert (np.abs(cs.cpu().numpy()[same] - ref.cos[same]) <= P.COS_RTOL * np.abs(ref.cos[same]) + P.COS_ATOL).all()
    assert np.allclose(probs.cpu().numpy(), ref.probs, rtol=1e-5, atol=1e-9)
    # the table really acts: against the unbiased gate some tokens change expert
    plain = oracle.gate(W.host_bits(x), sh.x_dtype, w.E)
    if w.T > 100 and w.E > 1:
        assert (plain.idx != ref.idx).any()


@pytest.mark.parametrize("kw", SHAPES)
@pytest.mark.parametrize("with_table", [False, True])
def test_probability_column_sums_inside_the_gate(P, kw, with_table):
    # L_aux = alpha n sum_i f_i P_i with P_i from the gate kernel's own partial sums: no probability matrix
    W, B, oracle = P.W, P.B, P.oracle
    w, dev, x, src, sh, idx, gw, cs = _setup(P, kw)
    table = np.random.default_rng(18).uniform(-0.05, 0.05, (sh.D, w.E)).astype(np.float32) if with_table else None
    eps = None if table is None else torch.as_tensor(table, device=dev)
    p_part = torch.full((B.GATE_PARTIAL_ROWS, w.E), float("nan"), device=dev)
    rows = B.locmoe_gate_ex(sh, x, idx, gw, cs, eps=eps, src_dev=src if with_table else None, p_part=p_part)
    assert 1 <= rows <= B.GATE_PARTIAL_ROWS
    load = torch.bincount(idx.long(), minlength=w.E).to(torch.int32)
    f = torch.empty(w.E, device=dev); Pm = torch.empty(w.E, device=dev); loss = torch.empty(1, device=dev)
    B.locmoe_aux_loss_partial(sh, p_part, rows, load, 0.01, f, Pm, loss)
    torch.cuda.synchronize()
    assert not torch.isnan(p_part[:rows]).any() and torch.isnan(p_part[rows:]).all()
    if with_table:
        ref = oracle.gate_per_source(W.host_bits(x), sh.x_dtype, w.E, table, src.cpu().numpy(), want_probs=True)
    else:
        ref = oracle.gate(W.host_bits(x), sh.x_dtype, w.E, want_probs=True)
    L, f_o, P_o = oracle.aux_loss(idx.cpu().numpy(), ref.probs, 0.01)
    assert np.allclose(Pm.cpu().numpy(), P_o, rtol=1e-5, atol=0)
    assert np.allclose(f.cpu().numpy(), f_o, rtol=1e-6, atol=0)
    assert abs(loss.item() - L) <= 1e-5 * L
    assert abs(float(Pm.double().sum()) - 1.0) < 1e-5
    # the other outputs are those of the plain gate, and a second run gives the same bits (fixed summation order)
    idx2 = torch.empty_like(idx); gw2 = torch.empty_like(gw); cs2 = torch.empty_like(cs)
    if not with_table:
        B.locmoe_gate(sh, x, None, idx2, gw2, cs2, None)
        assert torch.equal(idx, idx2) and torch.equal(gw, gw2) and torch.equal(cs, cs2)
    p2 = torch.zeros_like(p_part)
    assert B.locmoe_gate_ex(sh, x, idx2, gw2, cs2, eps=eps, src_dev=src if with_table else None, p_part=p2) == rows
    torch.cuda.synchronize()
    assert torch.equal(p2[:rows], p_part[:rows])


def test_gate_ex_rejects_a_source_array_without_a_table(P):
    import ctypes as C
    B = P.B
    sh = B.make_shape(64, 64, 8, 1, 2, B.BF16)
    one = C.c_void_p(256)
    opts = B.GateOpts(None, 256, None, None, 0)
    assert B._lib.locmoe_gate_ex(C.byref(sh), one, C.byref(opts), one, one, one, None) == -1
    assert B._lib.locmoe_gate_ex(C.byref(sh), one, None, one, one, one, None) == -1
    assert B._lib.locmoe_aux_loss_partial(C.byref(sh), one, 0, one, 0.01, one, one, one, None) == -2
