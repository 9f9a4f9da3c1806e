"""Top-k variant on the GPU against the oracle: choices, scores, routing of the K * T virtual tokens, buffer, combine."""
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


CASES = [
    dict(T=3000, H=512, E=16, n_nodes=2, dev_per_node=4, dtype="bf16", K=2, cf=1.0, layout=0),
    dict(T=2000, H=768, E=8, n_nodes=2, dev_per_node=2, dtype="f32", K=3, cf=1.25, layout=1),
    dict(T=2500, H=5120, E=64, n_nodes=8, dev_per_node=8, dtype="bf16", K=2, cf=1.0, layout=0, src="mod"),
    dict(T=900, H=256, E=4, n_nodes=1, dev_per_node=2, dtype="f32", K=4, cf=0.5, layout=1),      # K = E
    dict(T=1200, H=512, E=16, n_nodes=2, dev_per_node=4, dtype="bf16", K=1, cf=1.0, layout=0),   # K = 1: the top-1 path
]


@pytest.mark.parametrize("case", CASES)
def test_topk_path_against_oracle(P, case):
    W, B, oracle = P.W, P.B, P.oracle
    case = dict(case)
    K, cf, layout = case.pop("K"), case.pop("cf"), case.pop("layout")
    dev = torch.device("cuda:0")
    w = W.Workload(name="topk", config=6, tokens="normal", **{"src": "uniform", **case})
    x, src = W.make_tokens(w, dev), W.make_src(w, dev)
    D = w.n_nodes * w.dev_per_node
    sh = B.make_shape(w.T, w.H, w.E, w.n_nodes, w.dev_per_node, x.dtype, layout)
    Ca = B.conventional_capacity(K * w.T, D, w.E, cf)
    r = B.router_forward_topk(sh, x, src, K, Ca, B.CapacityRule(1.0, cf, -1.0, 0, 0))
    torch.cuda.synchronize()
    xh = W.host_bits(x)
    idx_o, R_o, gap = oracle.gate_topk(xh, sh.x_dtype, w.E, K)

    # choices and scores: identical except where the logits involved are within 1e-6 of a tie
    idx_g = r["idx_k"].cpu().numpy()
    w_g = r["w_k"].cpu().numpy().astype(np.float64)
    differs = (idx_g != idx_o).any(0)
    assert differs.sum() <= (gap < 1e-6).sum() and not (differs & (gap >= 1e-6)).any()
    same = idx_g == idx_o
    assert np.allclose(w_g[same], R_o[same], rtol=1e-5, atol=1e-9)

    # capacity counts K * T assignments
    cap = B.locmoe_capacity_read(r["cap_dev"])
    assert cap.C_local == int(np.ceil(cf * K * w.T / (D * w.E))) == Ca

    # route of the virtual tokens: the oracle's own choices, with the GPU's taken at the near-tie tokens verified above
    src_h = src.cpu().numpy()
    idx_in = np.where(differs[None, :], idx_g, idx_o)
    ref = oracle.route(idx_in.reshape(-1), np.tile(src_h, K), w.E, w.n_nodes, w.dev_per_node, cap.C_local, Ca, layout)
    assert np.array_equal(r["slot"].cpu().numpy().reshape(-1), ref.slot)
    assert np.array_equal(r["pos"].cpu().numpy().reshape(-1), ref.pos)
    assert np.array_equal(r["counts"].cpu().numpy().reshape(D, w.E), ref.counts)
    inv_g = r["inv"].cpu().numpy()
    assert np.array_equal(inv_g, np.where(ref.inv >= 0, ref.inv % w.T, -1))
    if K > 1:
        # a first choice is never displaced by a second one: within a (source, expert) queue first choices come first
        slot_k = ref.slot.reshape(K, w.T)
        pos_k = ref.pos.reshape(K, w.T)
        key0, key1 = src_h * w.E + idx_g[0], src_h * w.E + idx_g[1]
        n_first = np.bincount(key0, minlength=D * w.E)
        assert (pos_k[1] >= n_first[key1]).all()
        assert (slot_k < 0).any()

    # buffer: every assignment's row is a copy of its token
    rows = D * w.E * Ca
    want_buf = oracle.dispatch(np.tile(xh, (K, 1)), sh.x_dtype, ref.slot, rows)
    assert np.array_equal(W.host_bits(r["buf"]), want_buf)

    # combine over the K choices, one rounding
    R_use = np.where(same, R_o, w_g)
    want_out = oracle.combine_topk(want_buf, sh.x_dtype, ref.slot.reshape(K, w.T), R_use)
    P._out_close(W.host_bits(r["out"]), want_out, sh.x_dtype)


def test_topk_combine_with_random_fp32_expert_outputs(P):
    W, B, oracle = P.W, P.B, P.oracle
    dev = torch.device("cuda:0")
    w = W.Workload(name="topk", config=6, tokens="normal", src="uniform", T=1500, H=1024, E=16, n_nodes=2, dev_per_node=4, dtype="bf16")
    x, src = W.make_tokens(w, dev), W.make_src(w, dev)
    sh = B.make_shape(w.T, w.H, w.E, 2, 4, x.dtype, 1)
    K, Ca = 2, B.conventional_capacity(2 * w.T, 8, w.E, 1.0)
    gen = torch.Generator(device=dev).manual_seed(99)
    y = torch.randn(8 * w.E * Ca, w.H, generator=gen, device=dev)
    r = B.router_forward_topk(sh, x, src, K, Ca, B.CapacityRule(1.0, 1.0, -1.0, 0, 0), y=y)
    torch.cuda.synchronize()
    yh, slot_h, wk_h = y.cpu().numpy(), r["slot"].cpu().numpy(), r["w_k"].cpu().numpy().astype(np.float64)
    want = oracle.combine_topk(yh, oracle.F32, slot_h, wk_h)
    # two terms of opposite sign can cancel: the fp32 accumulation error scales with the terms, not with the sum, so
    # the bound is half a bf16 ulp of the result plus two fp32 ulps of the sum of the terms' magnitudes
    mag = oracle.combine_topk(np.abs(yh), oracle.F32, slot_h, wk_h)
    got = oracle.bf16_bits_to_f64(W.host_bits(r["out"]))
    err = np.abs(got - want)
    assert err.max() <= P.BF16_OUT_ATOL
    assert (err <= 1.02 * 2.0 ** -8 * np.abs(want) + 2.0 ** -22 * mag + 2.0 ** -126).all()
