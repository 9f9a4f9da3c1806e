"""Dispatch / combine fused with the exchange (peer stores and loads), with the ranks emulated on one GPU.

Every emulated rank is a separate set of calls on its own tokens (those of its logical source devices) and writes
through the same pointer table the multi-GPU run would use; here all "peer" buffers live on the one GPU.  No kernel
waits on another, so running the ranks one after the other is the same computation.  The concatenated receive
buffers must equal the oracle's receive-side buffer of the whole batch bit for bit."""
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
    dict(T=3000, H=512, E=16, n_nodes=2, dev_per_node=4, dtype="bf16", world=2),
    dict(T=3000, H=512, E=16, n_nodes=2, dev_per_node=4, dtype="f32", world=4),
    dict(T=2500, H=1024, E=32, n_nodes=4, dev_per_node=2, dtype="bf16", world=8),
    dict(T=1500, H=5120, E=64, n_nodes=8, dev_per_node=8, dtype="bf16", world=4, src="mod"),
    dict(T=700, H=256, E=8, n_nodes=2, dev_per_node=2, dtype="f32", world=1),
]


@pytest.mark.parametrize("case", CASES)
def test_emulated_ranks_match_the_oracles_receive_buffer(P, case):
    from paper_2401_13920_b200 import sharding
    W, B, oracle = P.W, P.B, P.oracle
    case = dict(case)
    world = case.pop("world")
    dev = torch.device("cuda:0")
    w = W.Workload(name="peer", config=7, tokens="normal", **{"src": "uniform", **case})
    x, src = W.make_tokens(w, dev), W.make_src(w, dev)
    D = w.n_nodes * w.dev_per_node
    cf = 1.0
    Ca = B.conventional_capacity(w.T, D, w.E, cf)
    rule = B.CapacityRule(1.0, cf, -1.0, 0, 0)

    # the whole batch on one GPU gives the capacity record every rank uses (a multi-GPU run all-reduces the minima)
    sh_g = B.make_shape(w.T, w.H, w.E, w.n_nodes, w.dev_per_node, x.dtype, B.LAYOUT_RECV)
    st_g = B.make_router(sh_g, Ca, rule, dev)
    B.router_forward(st_g, x, src)
    torch.cuda.synchronize()
    cap = B.locmoe_capacity_read(st_g.cap_dev)
    src_h = src.cpu().numpy()
    # the oracle's own arg-max indices; the GPU's pick only at tokens whose two best logits are within 1e-6
    g = oracle.gate(W.host_bits(x), sh_g.x_dtype, w.E)
    idx_gpu = st_g.idx.cpu().numpy()
    flip = idx_gpu != g.idx
    assert (g.gap[flip] < 1e-6).all()
    idx_h = np.where(flip, idx_gpu, g.idx)
    ref = oracle.route(idx_h, src_h, w.E, w.n_nodes, w.dev_per_node, cap.C_local, Ca, B.LAYOUT_RECV)
    rows = D * w.E * Ca
    want = oracle.dispatch(W.host_bits(x), sh_g.x_dtype, ref.slot, rows)
    assert (ref.inv < 0).any() and (ref.slot < 0).any()

    rpp = rows // world
    sentinel = 1.5
    bufs = [torch.full((rpp, w.H), sentinel, dtype=x.dtype, device=dev) for _ in range(world)]
    ranks = []
    # phase 1 on every rank: gate and the per-expert minima of its own tokens; the minimum over the ranks (an
    # All-Reduce MIN in a multi-GPU run, sharding.global_capacity_inputs) gives the batch-wide delta
    pre = []
    for q in range(world):
        sel = sharding.shard_by_source(src_h, D, world, q)
        sel_d = torch.as_tensor(sel, device=dev)
        x_q, src_q = x[sel_d].contiguous(), src[sel_d].contiguous()
        sh_q = B.make_shape(len(sel), w.H, w.E, w.n_nodes, w.dev_per_node, x.dtype, B.LAYOUT_RECV)
        st_q = B.make_router(sh_q, Ca, rule, dev)
        B.locmoe_gate(sh_q, x_q, None, st_q.idx, st_q.gate_w, st_q.cos_sim, None)
        B.locmoe_capacity(sh_q, st_q.idx, st_q.cos_sim, rule, st_q.delta_e, st_q.theta_e, st_q.cap_dev, st_q.ws)
        pre.append((sel, sel_d, x_q, src_q, sh_q, st_q))
    torch.cuda.synchronize()
    delta = min(max(min(float(p[5].delta_e.min().item()) for p in pre), 0.0), 1.0)
    rule_g = B.CapacityRule(1.0, cf, delta, 0, w.T)
    for q in range(world):
        sel, sel_d, x_q, src_q, sh_q, st_q = pre[q]
        devs = sharding.devices_of_rank(D, world, q)
        B.locmoe_capacity(sh_q, st_q.idx, st_q.cos_sim, rule_g, st_q.delta_e, st_q.theta_e, st_q.cap_dev, st_q.ws)
        cap_q = B.locmoe_capacity_read(st_q.cap_dev)
        assert (cap_q.C_local, cap_q.C_expert, cap_q.delta, cap_q.ec_min) == (cap.C_local, cap.C_expert, cap.delta, cap.ec_min)
        B.locmoe_route(sh_q, st_q.idx, src_q, st_q.cap_dev, Ca, st_q.pos, st_q.slot, st_q.drop, st_q.inv, st_q.counts,
                       st_q.kept, st_q.send_counts, st_q.load, st_q.locality, st_q.status, st_q.ws)
        B.locmoe_dispatch_peer(sh_q, Ca, x_q, st_q.inv, st_q.slot, bufs, devs.start, devs.stop, True)
        torch.cuda.synchronize()
        assert np.array_equal(st_q.slot.cpu().numpy(), ref.slot[sel])       # local routing = the global one, restricted
        if q == 0 and world > 1:
            # rows that belong to other ranks' source devices have not been touched yet
            allb = torch.cat(bufs).float()
            untouched = (allb == sentinel).all(dim=1).cpu().numpy()
            src_of_row = _row_sources(rows, Ca, D, w.E // D, w.n_nodes, w.dev_per_node)
            mine = (src_of_row >= devs.start) & (src_of_row < devs.stop)
            assert np.array_equal(untouched, ~mine)
        ranks.append((sel, sel_d, sh_q, st_q))

    got = torch.cat(bufs)
    assert np.array_equal(W.host_bits(got), want), "receive buffers differ from the oracle's"

    # combine through peer loads: identity experts, so y = the receive buffers themselves
    ydt = B.dtype_code(x.dtype)
    for sel, sel_d, sh_q, st_q in ranks:
        out = torch.empty(len(sel), w.H, dtype=x.dtype, device=dev)
        B.locmoe_combine_peer(sh_q, Ca, bufs, ydt, st_q.slot, st_q.gate_w, out)
        torch.cuda.synchronize()
        R = np.where(g.idx[sel] == st_q.idx.cpu().numpy(), g.R[sel], st_q.gate_w.cpu().numpy().astype(np.float64))
        ref_out = oracle.combine(want, sh_g.x_dtype, ref.slot[sel], R)
        P._out_close(W.host_bits(out), ref_out, sh_g.x_dtype)


def _row_sources(rows, C, D, Ed, N, Dn):
    """Source device of every receive-layout row, from the layout's definition (written out independently)."""
    r = np.arange(rows) // C
    e, rho = r // D, r % D
    a = e // Ed
    return ((a // Dn + rho // Dn) % N) * Dn + (a % Dn + rho % Dn) % Dn


def test_peer_calls_reject_bad_arguments(P):
    B = P.B
    dev = torch.device("cuda:0")
    sh = B.make_shape(64, 64, 8, 2, 2, torch.float32, B.LAYOUT_SEND)
    x = torch.zeros(64, 64, device=dev)
    inv = torch.full((4 * 8 * 4,), -1, dtype=torch.int32, device=dev)
    slot = torch.full((64,), -1, dtype=torch.int32, device=dev)
    buf = torch.zeros(4 * 8 * 4, 64, device=dev)
    with pytest.raises(B.LocMoEError):            # send-side layout
        B.locmoe_dispatch_peer(sh, 4, x, inv, slot, [buf], 0, 4)
    sh = B.make_shape(64, 64, 8, 2, 2, torch.float32, B.LAYOUT_RECV)
    with pytest.raises(B.LocMoEError):            # three peers do not divide four devices
        B.locmoe_dispatch_peer(sh, 4, x, inv, slot, [buf, buf, buf], 0, 4)
    with pytest.raises(B.LocMoEError):            # source range outside the map
        B.locmoe_dispatch_peer(sh, 4, x, inv, slot, [buf], 0, 5)


@pytest.mark.parametrize("with_ffn", [False, True])
def test_single_rank_peer_layer_equals_the_layer_call(P, with_ffn):
    # with one rank the fused-exchange sequence must reproduce locmoe_moe_layer bit for bit
    from paper_2401_13920_b200 import exchange, sharding
    W, B = P.W, P.B
    dev = torch.device("cuda:0")
    w = W.CONFIGS[5].scaled(4096)
    F = 512
    x, src = W.make_tokens(w, dev), W.make_src(w, dev)
    sh = B.make_shape(w.T, w.H, w.E, w.n_nodes, w.dev_per_node, x.dtype, B.LAYOUT_RECV)
    rule = B.CapacityRule(1.0, 1.0, -1.0, 0, 0)
    Ca = B.conventional_capacity(w.T, sh.D, w.E, 1.0)
    w_in = w_out = None
    if with_ffn:
        w_in, w_out = W.make_expert_weights(w, F, dev)
    # reference: the one-call layer
    st = B.make_router(sh, Ca, rule, dev)
    h1 = torch.empty(st.rows, F, dtype=torch.bfloat16, device=dev)
    y = torch.empty(st.rows, w.H, dtype=torch.bfloat16, device=dev)
    want = torch.empty(w.T, w.H, dtype=x.dtype, device=dev)
    B.locmoe_moe_layer(sh, x, src, None, rule, Ca, F, w_in, w_out, B.layer_buffers(st, h1, y), want)
    torch.cuda.synchronize()
    # the per-rank sequence with peer stores / loads
    st2 = B.make_router(sh, Ca, rule, dev)
    recv = exchange.PeerBuffers(st.rows, w.H, x.dtype, dev)
    yb = exchange.PeerBuffers(st.rows, w.H, torch.bfloat16, dev) if with_ffn else recv
    recv.local.fill_(3.0)
    h1b = torch.empty(st.rows, F, dtype=torch.bfloat16, device=dev)
    got = torch.empty(w.T, w.H, dtype=x.dtype, device=dev)
    exchange.peer_layer_forward(B, sharding, sh, Ca, rule, x, src, recv, yb, st2, w_in, w_out, F, h1b, out=got)
    torch.cuda.synchronize()
    assert B.locmoe_device_flags() == 0
    assert torch.equal(st2.slot, st.slot) and torch.equal(recv.local.view(torch.int16), st.buf.view(torch.int16))
    assert torch.equal(got.view(torch.int16), want.view(torch.int16))


@pytest.mark.parametrize("slices", [2, 8])
def test_sliced_overlap_of_exchange_and_experts_equals_the_unsliced_pass(P, slices):
    # the receive buffer filled expert block by expert block (windowed peer stores), the experts of a block running
    # on a second stream while the next block is stored: bit for bit the unsliced layer pass
    from paper_2401_13920_b200 import exchange, sharding
    W, B = P.W, P.B
    dev = torch.device("cuda:0")
    w = W.CONFIGS[5].scaled(6000)
    F = 768
    x, src = W.make_tokens(w, dev), W.make_src(w, dev)
    sh = B.make_shape(w.T, w.H, w.E, w.n_nodes, w.dev_per_node, x.dtype, B.LAYOUT_RECV)
    rule = B.CapacityRule(1.0, 1.0, -1.0, 0, 0)
    Ca = B.conventional_capacity(w.T, sh.D, w.E, 1.0)
    w_in, w_out = W.make_expert_weights(w, F, dev)
    outs = []
    for S in (1, slices):
        st = B.make_router(sh, Ca, rule, dev, with_buffer=False)
        recv = exchange.PeerBuffers(sh.D * w.E * Ca, w.H, x.dtype, dev)
        yb = exchange.PeerBuffers(sh.D * w.E * Ca, w.H, torch.bfloat16, dev)
        recv.local.fill_(3.0)
        yb.local.fill_(5.0)
        h1 = torch.empty(sh.D * w.E * Ca, F, dtype=torch.bfloat16, device=dev)
        got = torch.empty(w.T, w.H, dtype=x.dtype, device=dev)
        exchange.peer_layer_forward(B, sharding, sh, Ca, rule, x, src, recv, yb, st, w_in, w_out, F, h1, out=got, slices=S,
                                    ffn_stream=torch.cuda.Stream(dev))
        torch.cuda.synchronize()
        assert B.locmoe_device_flags() == 0
        outs.append((recv.local.clone(), yb.local.clone(), got.clone(), st.slot.clone()))
    a, b = outs
    assert int((a[3] < 0).sum()) > 0 and int((a[3] >= 0).sum()) > 0
    for u, v in zip(a, b):
        assert torch.equal(u.view(torch.int16) if u.dtype == torch.bfloat16 else u, v.view(torch.int16) if v.dtype == torch.bfloat16 else v)


def test_windowed_peer_dispatch_touches_only_its_window(P):
    W, B = P.W, P.B
    dev = torch.device("cuda:0")
    w = W.Workload(name="win", config=7, T=2000, H=256, E=8, n_nodes=2, dev_per_node=2, dtype="bf16", tokens="normal", src="uniform")
    x, src = W.make_tokens(w, dev), W.make_src(w, dev)
    sh = B.make_shape(w.T, w.H, w.E, 2, 2, x.dtype, B.LAYOUT_RECV)
    Ca = B.conventional_capacity(w.T, 4, w.E, 1.0)
    st = B.make_router(sh, Ca, B.CapacityRule(1.0, 1.0, -1.0, 0, 0), dev)
    B.router_forward(st, x, src)                       # st.buf: the whole receive-side buffer
    rows = st.rows
    halves = [torch.full((rows // 2, w.H), 9.0, dtype=x.dtype, device=dev) for _ in range(2)]    # two "peers"
    lo, hi = rows // 8, rows // 4                       # a window inside each peer's slice
    B.locmoe_dispatch_peer(sh, Ca, x, st.inv, st.slot, halves, 0, 4, True, window=(lo, hi))
    torch.cuda.synchronize()
    for q in range(2):
        want = torch.full_like(halves[q], 9.0)
        want[lo:hi] = st.buf[q * (rows // 2) + lo:q * (rows // 2) + hi]
        assert torch.equal(halves[q].view(torch.int16), want.view(torch.int16))
