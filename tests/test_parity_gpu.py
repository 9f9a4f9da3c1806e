"""GPU parity: the CUDA path, called through the C-ABI binding, against the CPU
oracle on the same seeded inputs (stage by stage, see tests/parity.py)."""
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


def _wl(P, **kw):
    base = dict(name="case", config=9, T=1000, H=256, E=8, n_nodes=2, dev_per_node=2, dtype="bf16",
                tokens="normal", src="uniform")
    base.update(kw)
    return P.W.Workload(**base)


# ---- the five configurations at sizes the oracle covers element by element ----

@pytest.mark.parametrize("layout", [0, 1])
def test_config1_tiny_full_size(P, layout):
    rep = P.run_staged(P.W.CONFIGS[1], 1.0, layout=layout, full=True)
    assert rep["C_local"] == 64 and 0.02 < rep["drop_frac"] < 0.10


@pytest.mark.parametrize("cfg,T", [(2, 6000), (3, 8229), (5, 7001)])
def test_configs_scaled_full_compare(P, cfg, T):
    rep = P.run_staged(P.W.CONFIGS[cfg].scaled(T), 1.0, full=True)
    assert rep["status"] == 0
    # no near-tie was taken differently here: every expected value came from the oracle's own chain
    assert rep["oracle_chain_only"]


@pytest.mark.parametrize("mult", [1.0, 1.25, 2.0])
def test_config4_scaled_capacity_multipliers_random_fp32_expert_out(P, mult):
    # group width 20 bf16 (40 bytes): 16-byte vectors straddle group boundaries
    rep = P.run_staged(P.W.CONFIGS[4].scaled(5003), mult, full=True, y_random=True)
    assert rep["C_local"] == int(np.ceil(mult * 5003 / 65536))


# ---- full sizes, in the launch configuration the bench times; outputs sampled ----

@pytest.mark.parametrize("cfg", [2, 5, 3])
def test_configs_full_size_sampled(P, cfg):
    w = P.W.CONFIGS[cfg]
    rep = P.run_staged(w, 1.0, full=False, n_sample=1024)
    assert rep["C_local"] == w.T // (w.D * w.E)
    if cfg == 3:
        assert rep["drop_frac"] > 0.3     # the Zipf mixture forces imbalance and drops
    else:
        assert 0.03 < rep["drop_frac"] < 0.15


@pytest.mark.parametrize("mult,C_local", [(1.0, 16), (1.25, 20), (2.0, 32)])
def test_config4_full_size_sampled(P, mult, C_local):
    # the capacity multipliers of the large-batch configuration at its full size (both knobs); up to 86 GB on the device
    w = P.W.CONFIGS[4]
    rep = P.run_staged(w, mult, full=False, n_sample=1024, y_random=True)
    assert rep["C_local"] == C_local and rep["oracle_chain_only"]
    if mult == 1.0:
        assert 0.05 < rep["drop_frac"] < 0.15
    elif mult == 1.25:
        assert 0.005 < rep["drop_frac"] < 0.05
    else:
        assert rep["drop_frac"] < 1e-3
    torch.cuda.empty_cache()


# ---- the large-batch variants (multi-kernel capacity, prescanned route histograms) forced at small sizes ----

@pytest.fixture
def grid_path(monkeypatch):
    monkeypatch.setenv("LOCMOE_PATH", "grid")


@pytest.mark.parametrize("cfg,T", [(1, 4096), (2, 70001), (3, 8229), (4, 5003), (5, 7001)])
def test_grid_path_configs(P, grid_path, cfg, T):
    rep = P.run_staged(P.W.CONFIGS[cfg].scaled(T), 1.0, full=True, y_random=cfg == 4)
    assert rep["status"] == 0


@pytest.mark.parametrize("kw", [
    dict(T=1, H=64, E=4, n_nodes=1, dev_per_node=2),
    dict(T=513, H=1024, E=512, n_nodes=4, dev_per_node=8),
    dict(T=4097, H=2048, E=2048, n_nodes=8, dev_per_node=8),
])
def test_grid_path_shapes(P, grid_path, kw):
    P.run_staged(_wl(P, **kw), 1.0, layout=1, full=True)


@pytest.mark.parametrize("cfg,T", [(2, 3001), (4, 2999)])
def test_general_gate_kernel_on_the_common_shapes(P, monkeypatch, cfg, T):
    # the common bf16 shapes normally take the specialised gate kernel; LOCMOE_GATE=general forces the general one
    monkeypatch.setenv("LOCMOE_GATE", "general")
    P.run_staged(P.W.CONFIGS[cfg].scaled(T), 1.0, full=True)


@pytest.mark.parametrize("H,E", [(4096, 64), (7168, 256), (4096, 32)])
def test_specialised_gate_kernel_other_shapes(P, H, E):
    P.run_staged(_wl(P, T=1500, H=H, E=E, n_nodes=2, dev_per_node=4), 1.0, full=True)


def test_bulk_copy_dispatch_variant(P, monkeypatch):
    # the TMA (cp.async.bulk) dispatch kernel: whole rows, split rows (> 16 KB), zero rows
    monkeypatch.setenv("LOCMOE_DISPATCH", "tma")
    P.run_staged(P.W.CONFIGS[2].scaled(6000), 1.25, full=True)
    P.run_staged(_wl(P, T=300, H=16384, E=8, n_nodes=2, dev_per_node=2, dtype="f32"), 2.0, full=True)
    P.run_staged(P.W.CONFIGS[1], 1.0, layout=1, full=True)


def test_warp_per_row_dispatch_variant(P, monkeypatch):
    # the warp-per-row dispatch kernel (the default is the flat (row, vector) mapping)
    monkeypatch.setenv("LOCMOE_DISPATCH", "vec")
    P.run_staged(P.W.CONFIGS[2].scaled(6000), 1.25, full=True)
    P.run_staged(_wl(P, T=1500, H=1000, E=8, n_nodes=2, dev_per_node=2, dtype="f32"), 0.5, full=True)
    P.run_staged(P.W.CONFIGS[1], 1.0, layout=1, full=True)


# ---- gate, capacity and route as ONE call chain (the gate kernel takes the route stage's first pass) ----

@pytest.mark.parametrize("cfg,T", [(1, 4096), (2, 6000), (3, 8229), (4, 5003), (5, 7001)])
@pytest.mark.parametrize("layout", [0, 1])
def test_gate_route_call_configs(P, cfg, T, layout):
    rep = P.run_staged(P.W.CONFIGS[cfg].scaled(T), 1.0, layout=layout, full=True, y_random=cfg == 4, fused="gate")
    assert rep["status"] == 0


@pytest.mark.parametrize("kw", [
    dict(T=1, H=64, E=4, n_nodes=1, dev_per_node=2),
    dict(T=31, H=64, E=1, n_nodes=1, dev_per_node=1),
    dict(T=777, H=60, E=4, n_nodes=1, dev_per_node=4, dtype="f32"),     # general vector gate kernel
    dict(T=777, H=36, E=4, n_nodes=2, dev_per_node=2),                  # scalar gate kernel
    dict(T=513, H=1024, E=512, n_nodes=4, dev_per_node=8),
    dict(T=3000, H=4096, E=2048, n_nodes=1, dev_per_node=1),
    dict(T=4097, H=2048, E=2048, n_nodes=8, dev_per_node=8),            # three radix passes
    dict(T=300, H=16384, E=16384, n_nodes=1, dev_per_node=1),           # > 8192 experts
])
def test_gate_route_call_shapes(P, kw):
    P.run_staged(_wl(P, **kw), 1.0, layout=1, full=True, fused="gate")


def test_gate_route_call_grid_path_and_full_size(P, monkeypatch):
    rep = P.run_staged(P.W.CONFIGS[2], 1.0, full=False, n_sample=512, fused="gate")
    assert rep["C_local"] == 16
    rep = P.run_staged(P.W.CONFIGS[3], 1.0, full=False, n_sample=512, fused="gate")
    assert rep["drop_frac"] > 0.3
    monkeypatch.setenv("LOCMOE_PATH", "grid")
    P.run_staged(P.W.CONFIGS[2].scaled(70001), 1.0, full=True, fused="gate")


def test_gate_route_call_with_bias_bad_sources_and_clamp(P):
    import numpy as np
    W, B = P.W, P.B
    w = _wl(P, T=2000, H=512, E=16, n_nodes=2, dev_per_node=4)
    P.run_staged(w, 1.0, eps=np.linspace(-0.05, 0.05, 16).astype(np.float32), full=True, fused="gate")
    rep = P.run_staged(P.W.CONFIGS[1], 2.0, C_alloc=40, full=True, fused="gate")
    assert rep["status"] & 1
    # a token with an impossible source device is dropped and flagged by the gate kernel's hook
    dev = torch.device("cuda:0")
    x, src = W.make_tokens(w, dev), W.make_src(w, dev).clone()
    src[5] = 99
    src[700] = -3
    sh = B.make_shape(w.T, w.H, w.E, 2, 4, x.dtype)
    st = B.make_router(sh, 20, B.CapacityRule(1.0, 1.0, -1.0, 0, 0), dev)
    B.router_forward(st, x, src, fused="gate")
    torch.cuda.synchronize()
    ref = B.make_router(sh, 20, B.CapacityRule(1.0, 1.0, -1.0, 0, 0), dev)
    B.router_forward(ref, x, src, fused=False)
    torch.cuda.synchronize()
    assert st.status.item() == ref.status.item() == 2
    for name in ("pos", "slot", "drop", "inv", "counts", "kept", "send_counts", "load", "locality", "idx"):
        assert torch.equal(getattr(st, name), getattr(ref, name)), name
    assert torch.equal(st.out.view(torch.int16), ref.out.view(torch.int16))
    assert st.slot[5].item() == -1 and st.slot[700].item() == -1


# ---- capacity and route as two separate calls (the default path runs them as the one fused call) ----

@pytest.mark.parametrize("cfg,T", [(1, 4096), (2, 6000), (3, 8229), (4, 5003), (5, 7001)])
def test_separate_capacity_and_route_calls(P, cfg, T):
    rep = P.run_staged(P.W.CONFIGS[cfg].scaled(T), 1.0, full=True, y_random=cfg == 4, fused=False)
    assert rep["status"] == 0


@pytest.mark.parametrize("kw", [
    dict(T=1, H=64, E=4, n_nodes=1, dev_per_node=2),
    dict(T=31, H=64, E=1, n_nodes=1, dev_per_node=1),
    dict(T=513, H=1024, E=512, n_nodes=4, dev_per_node=8),
    dict(T=4097, H=2048, E=2048, n_nodes=8, dev_per_node=8),
])
def test_separate_calls_shapes(P, kw):
    P.run_staged(_wl(P, **kw), 1.0, layout=1, full=True, fused=False)


def test_separate_calls_grid_path(P, grid_path):
    P.run_staged(P.W.CONFIGS[2].scaled(70001), 1.0, full=True, fused=False)


def test_separate_calls_full_size_config2(P):
    rep = P.run_staged(P.W.CONFIGS[2], 1.0, full=False, n_sample=512, fused=False)
    assert rep["C_local"] == 16


# ---- edge cases and degenerate inputs ----

@pytest.mark.parametrize("kw", [
    dict(T=1, H=64, E=4, n_nodes=1, dev_per_node=2),
    dict(T=31, H=64, E=1, n_nodes=1, dev_per_node=1),                   # one expert: R = 1
    dict(T=777, H=60, E=4, n_nodes=1, dev_per_node=4, dtype="f32"),     # odd group width 15 (unit = 1 element)
    dict(T=777, H=16, E=8, n_nodes=2, dev_per_node=2),                  # group width 2
    dict(T=777, H=36, E=4, n_nodes=2, dev_per_node=2),                  # rows of 72 bytes: scalar path
    dict(T=513, H=1024, E=512, n_nodes=4, dev_per_node=8),              # many experts, Ed = 16
    dict(T=2049, H=2048, E=8, n_nodes=2, dev_per_node=4, dtype="f32"),  # group spans whole warp iterations
    dict(T=3000, H=4096, E=2048, n_nodes=1, dev_per_node=1),            # > 1024 keys on a single device
    dict(T=4097, H=2048, E=2048, n_nodes=8, dev_per_node=8),            # 131072 keys: three radix passes; g = 1
    dict(T=300, H=16384, E=16384, n_nodes=1, dev_per_node=1),           # > 8192 experts: minima by global atomics,
                                                                        # capacity and route not fused
])
@pytest.mark.parametrize("layout", [0, 1])
def test_shapes(P, kw, layout):
    P.run_staged(_wl(P, **kw), 1.0, layout=layout, full=True)


def test_literal_minimum_mode_one_slot_per_pair(P):
    # c_f = 0: capacity = ceil(Theorem 1's minimum) = 1 slot per (source, expert) pair
    rep = P.run_staged(P.W.CONFIGS[2].scaled(20000), 0.0, min_mult=1.0, C_alloc=1, full=True)
    assert rep["C_local"] == 1 and rep["drop_frac"] > 0.7


def test_minimum_binds_on_aligned_tokens(P):
    # tokens pushed along their expert's gating direction: large delta, Theorem 1's minimum exceeds T / n
    w = _wl(P, T=4096, H=1024, E=8, n_nodes=2, dev_per_node=4, dtype="f32", tokens="zipf_mixture", config=8)
    rep = P.run_staged(w, 0.5, min_mult=1.0, delta_override=0.134, C_alloc=600, full=True)
    assert rep["C_expert"] == 4096 and rep["C_local"] == 512


@pytest.mark.parametrize("form", [1, 2])
def test_bound_forms_with_the_papers_delta(P, form):
    rep = P.run_staged(P.W.CONFIGS[2].scaled(3000), 1.0, delta_override=0.03, bound_form=form, full=True)
    assert rep["delta"] == 0.03


def test_capacity_clamped_to_the_allocation(P):
    rep = P.run_staged(P.W.CONFIGS[1], 2.0, C_alloc=40, full=True)
    assert rep["status"] & 1 and rep["C_local"] == 128


def test_bias_and_probs(P):
    W, B = P.W, P.B
    w = _wl(P, T=2000, H=512, E=16, n_nodes=2, dev_per_node=4)
    eps = np.linspace(-0.05, 0.05, 16).astype(np.float32)
    P.run_staged(w, 1.0, eps=eps, full=True)
    dev = torch.device("cuda:0")
    x = W.make_tokens(w, dev)
    sh = B.make_shape(w.T, w.H, w.E, 2, 4, x.dtype)
    idx = torch.empty(w.T, dtype=torch.int32, device=dev)
    gw = torch.empty(w.T, device=dev)
    cs = torch.empty(w.T, device=dev)
    probs = torch.empty(w.T, w.E, device=dev)
    B.locmoe_gate(sh, x, torch.as_tensor(eps, device=dev), idx, gw, cs, probs)
    ref = P.oracle.gate(W.host_bits(x), sh.x_dtype, w.E, eps=eps, want_probs=True)
    assert np.allclose(probs.cpu().numpy(), ref.probs, rtol=1e-5, atol=1e-9)
    assert torch.allclose(probs.sum(1), torch.ones(w.T, device=dev), atol=1e-5)


def test_bad_source_device_is_dropped_and_flagged(P):
    W, B = P.W, P.B
    w = _wl(P, T=1500, H=128, E=8, n_nodes=2, dev_per_node=2)
    dev = torch.device("cuda:0")
    x = W.make_tokens(w, dev)
    src = W.make_src(w, dev)
    src[7] = 99
    src[1200] = -3
    sh = B.make_shape(w.T, w.H, w.E, 2, 2, x.dtype)
    rule = B.CapacityRule(1.0, 1.0, -1.0, 0, 0)
    st = B.make_router(sh, 60, rule, dev)
    B.router_forward(st, x, src)
    torch.cuda.synchronize()
    cap = B.locmoe_capacity_read(st.cap_dev)
    ref = P.check_route(sh, st, src, cap)
    assert ref.status == 2 and ref.drop[7] == 1 and ref.pos[1200] == -1
    assert not st.out[7].any().item()


def test_non_finite_tokens_stay_local_to_their_rows(P):
    # infinities / NaNs in a few tokens: every other token's outputs are bit for bit those of the clean batch, the
    # poisoned tokens still get an expert index in range, and the routing stays a valid placement
    W, B = P.W, P.B
    dev = torch.device("cuda:0")
    for kw in (dict(T=3000, H=5120, E=64, n_nodes=8, dev_per_node=8), dict(T=2000, H=60, E=4, n_nodes=1, dev_per_node=4, dtype="f32")):
        w = _wl(P, **kw)
        x, src = W.make_tokens(w, dev), W.make_src(w, dev)
        sh = B.make_shape(w.T, w.H, w.E, w.n_nodes, w.dev_per_node, x.dtype)
        Ca = B.conventional_capacity(w.T, sh.D, w.E, 1.0)
        rule = B.CapacityRule(1.0, 1.0, 0.01, 0, 0)          # a fixed threshold: the capacity must not depend on the poison
        clean = B.make_router(sh, Ca, rule, dev)
        B.router_forward(clean, x, src)
        torch.cuda.synchronize()
        xp = x.clone()
        bad = [3, 700, w.T - 1]
        xp[3, 5] = float("inf")
        xp[700, 0] = float("nan")
        xp[w.T - 1, w.H - 1] = float("-inf")
        xp[w.T - 1, 1] = float("inf")
        st = B.make_router(sh, Ca, rule, dev)
        B.router_forward(st, xp, src)
        torch.cuda.synchronize()
        assert B.locmoe_device_flags() == 0
        good = torch.ones(w.T, dtype=torch.bool, device=dev)
        good[bad] = False
        for name in ("idx", "gate_w", "cos_sim"):
            assert torch.equal(getattr(st, name)[good], getattr(clean, name)[good]), name
        assert int(st.idx.min()) >= 0 and int(st.idx.max()) < w.E
        keep = st.slot >= 0
        assert len(torch.unique(st.slot[keep])) == int(keep.sum())                 # all slots distinct
        assert torch.equal(st.inv[st.slot[keep].long()], torch.nonzero(keep).flatten().to(torch.int32))
        assert int(st.kept.max()) <= B.locmoe_capacity_read(st.cap_dev).C_local
        assert int(st.kept.sum()) + int(st.drop.sum()) == w.T


def test_accumulate_adds_to_the_output(P):
    W, B = P.W, P.B
    w = _wl(P, T=900, H=256, E=8, n_nodes=2, dev_per_node=2, dtype="f32")
    dev = torch.device("cuda:0")
    x = W.make_tokens(w, dev)
    src = W.make_src(w, dev)
    sh = B.make_shape(w.T, w.H, w.E, 2, 2, x.dtype)
    st = B.make_router(sh, 20, B.CapacityRule(1.0, 1.0, -1.0, 0, 0), dev)
    B.router_forward(st, x, src)
    first = st.out.clone()
    B.locmoe_combine(sh, 20, st.buf, st.slot, st.gate_w, st.out, accumulate=True)
    torch.cuda.synchronize()
    ref = P.oracle.combine(W.host_bits(st.buf), B.F32, st.slot.cpu().numpy(), st.gate_w.double().cpu().numpy(),
                           prev=first.double().cpu().numpy())
    assert np.allclose(st.out.cpu().numpy(), ref, rtol=1e-5, atol=1e-6)


def test_round_trip_identity_experts_unit_scores(P):
    # combine(dispatch(x)) with R = 1 returns x bit for bit on kept tokens and 0 on dropped ones
    W, B = P.W, P.B
    w = P.W.CONFIGS[5].scaled(9000)
    dev = torch.device("cuda:0")
    x = W.make_tokens(w, dev)
    src = W.make_src(w, dev)
    sh = B.make_shape(w.T, w.H, w.E, w.n_nodes, w.dev_per_node, x.dtype)
    st = B.make_router(sh, 9, B.CapacityRule(1.0, 1.0, -1.0, 0, 0), dev)
    B.router_forward(st, x, src)
    ones = torch.ones(w.T, device=dev)
    B.locmoe_combine(sh, 9, st.buf, st.slot, ones, st.out)
    torch.cuda.synchronize()
    keep = st.slot >= 0
    assert 0 < int(keep.sum()) < w.T
    assert torch.equal(st.out[keep].view(torch.int16), x[keep].view(torch.int16))
    assert not st.out[~keep].any().item()


def test_route_is_deterministic(P):
    W, B = P.W, P.B
    w = P.W.CONFIGS[3].scaled(50000)
    dev = torch.device("cuda:0")
    x = W.make_tokens(w, dev)
    src = W.make_src(w, dev)
    sh = B.make_shape(w.T, w.H, w.E, w.n_nodes, w.dev_per_node, x.dtype)
    st = B.make_router(sh, 4, B.CapacityRule(1.0, 1.0, -1.0, 0, 0), dev)
    B.router_forward(st, x, src)
    torch.cuda.synchronize()
    a = [t.clone() for t in (st.pos, st.slot, st.inv, st.counts, st.send_counts, st.locality)]
    for _ in range(3):
        B.router_forward(st, x, src)
        torch.cuda.synchronize()
        for u, v in zip(a, (st.pos, st.slot, st.inv, st.counts, st.send_counts, st.locality)):
            assert torch.equal(u, v)


def test_host_router_pipeline_matches_device_path(P):
    # tokens in pinned host memory, three pipelined steps on different batches
    W, B = P.W, P.B
    dev = torch.device("cuda:0")
    w = P.W.CONFIGS[5].scaled(5000)
    sh = B.make_shape(w.T, w.H, w.E, w.n_nodes, w.dev_per_node, torch.bfloat16)
    rule = B.CapacityRule(1.0, 1.0, -1.0, 0, 0)
    Ca = B.conventional_capacity(w.T, sh.D, w.E, 1.0)
    hr = B.HostRouter(sh, Ca, rule, dev)
    st = B.make_router(sh, Ca, rule, dev)
    src = W.make_src(w, dev)
    srch = src.cpu().pin_memory()
    xs, outs = [], []
    for i in range(3):
        wi = W.Workload(**{**w.__dict__, "config": 5 + 10 * i})
        xs.append(W.make_tokens(wi, dev))
        outs.append(torch.empty(w.T, w.H, dtype=torch.bfloat16).pin_memory())
        hr.forward(xs[-1].cpu().pin_memory(), srch, outs[-1])
    hr.synchronize()
    for x, o in zip(xs, outs):
        ref = B.router_forward(st, x, src)
        torch.cuda.synchronize()
        assert torch.equal(o.view(torch.int16), ref.cpu().view(torch.int16))


def test_aux_loss_against_oracle(P):
    W, B = P.W, P.B
    dev = torch.device("cuda:0")
    w = P.W.CONFIGS[2].scaled(5000)
    x = W.make_tokens(w, dev)
    src = W.make_src(w, dev)
    sh = B.make_shape(w.T, w.H, w.E, w.n_nodes, w.dev_per_node, x.dtype)
    st = B.make_router(sh, 2, B.CapacityRule(1.0, 1.0, -1.0, 0, 0), dev)
    probs = torch.empty(w.T, w.E, device=dev)
    B.locmoe_gate(sh, x, None, st.idx, st.gate_w, st.cos_sim, probs)
    B.locmoe_capacity(sh, st.idx, st.cos_sim, st.rule, st.delta_e, st.theta_e, st.cap_dev, st.ws)
    B.locmoe_route(sh, st.idx, src, st.cap_dev, 2, st.pos, st.slot, st.drop, st.inv, st.counts, st.kept,
                   st.send_counts, st.load, st.locality, st.status, st.ws)
    f = torch.empty(w.E, device=dev); Pm = torch.empty(w.E, device=dev); loss = torch.empty(1, device=dev)
    B.locmoe_aux_loss(sh, probs, st.load, 0.01, f, Pm, loss, st.ws)
    torch.cuda.synchronize()
    g = P.oracle.gate(W.host_bits(x), sh.x_dtype, w.E, want_probs=True)
    assert (g.idx != st.idx.cpu().numpy()).sum() <= (g.gap < 1e-6).sum()
    L, f_o, P_o = P.oracle.aux_loss(st.idx.cpu().numpy(), g.probs, 0.01)
    assert np.allclose(f.cpu().numpy(), f_o, rtol=1e-6, atol=0)
    assert np.allclose(Pm.cpu().numpy(), P_o, rtol=1e-5, atol=0)
    assert abs(loss.item() - L) <= 1e-5 * L
    # deterministic: a second evaluation gives the same bits
    loss2 = torch.empty(1, device=dev)
    B.locmoe_aux_loss(sh, probs, st.load, 0.01, f, Pm, loss2, st.ws)
    torch.cuda.synchronize()
    assert loss2.item() == loss.item()


@pytest.mark.parametrize("cfg,T,level", [(2, 5000, 0), (2, 5000, 1), (3, 8229, 1), (1, 4096, 0)])
def test_locality_loss_against_oracle(P, cfg, T, level):
    # counts from the CUDA route stage (bit-exact against the oracle elsewhere) -> L_loc in fp64 on both sides
    W, B = P.W, P.B
    dev = torch.device("cuda:0")
    w = P.W.CONFIGS[cfg].scaled(T)
    x, src = W.make_tokens(w, dev), W.make_src(w, dev)
    sh = B.make_shape(w.T, w.H, w.E, w.n_nodes, w.dev_per_node, x.dtype)
    Ca = B.conventional_capacity(w.T, sh.D, w.E, 1.0)
    st = B.make_router(sh, Ca, B.CapacityRule(1.0, 1.0, -1.0, 0, 0), dev)
    B.router_forward(st, x, src)
    G = w.n_nodes if level else sh.D
    dc = torch.empty(G, w.E, device=dev)
    kl = torch.empty(G, dtype=torch.float64, device=dev)
    nt = torch.empty(G, dtype=torch.int64, device=dev)
    loss = torch.empty(1, dtype=torch.float64, device=dev)
    B.locmoe_loc_loss(sh, st.counts, level, 0.5, 1e-3, dc, kl, nt, loss)
    torch.cuda.synchronize()
    counts = st.counts.cpu().numpy()
    L, dc_o, kl_o = P.oracle.loc_loss(counts, w.E, w.n_nodes, w.dev_per_node, level=level, mu=0.5, smooth=1e-3)
    assert np.array_equal(nt.cpu().numpy(), counts.reshape(G, -1).sum(1))
    assert np.allclose(kl.cpu().numpy(), kl_o, rtol=1e-12, atol=1e-15)
    assert np.allclose(dc.cpu().numpy(), dc_o, rtol=1e-6, atol=0)
    assert abs(loss.item() - L) <= 1e-12 * abs(L) and L > 0
    loss2 = torch.empty(1, dtype=torch.float64, device=dev)
    B.locmoe_loc_loss(sh, st.counts, level, 0.5, 1e-3, dc, kl, nt, loss2)
    torch.cuda.synchronize()
    assert loss2.item() == loss.item()


@pytest.mark.parametrize("cfg,T,dtype_name", [(2, 20000, "bf16"), (1, 4096, "f32"), (3, 8229, "bf16")])
def test_cosine_histograms_against_oracle(P, cfg, T, dtype_name):
    # bins are decided in fp32 by the kernel and in fp64 by the oracle: a token whose cosine lies within 1e-6 of a
    # bin edge may fall on either side; everything else must agree exactly
    W, B = P.W, P.B
    dev = torch.device("cuda:0")
    w = P.W.CONFIGS[cfg].scaled(T)
    x = W.make_tokens(w, dev)
    sh = B.make_shape(w.T, w.H, w.E, w.n_nodes, w.dev_per_node, x.dtype)
    idx = torch.empty(w.T, dtype=torch.int32, device=dev)
    gw = torch.empty(w.T, device=dev); cs = torch.empty(w.T, device=dev)
    B.locmoe_gate(sh, x, None, idx, gw, cs, None)
    nb, lo, hi = 64, -0.125, 0.25
    he = torch.empty(nb, dtype=torch.int32, device=dev); hj = torch.empty(nb, dtype=torch.int32, device=dev)
    n = torch.empty(1, dtype=torch.int32, device=dev)
    e = int(torch.bincount(idx.long(), minlength=w.E).argmax())
    j = (e + 1) % w.E
    B.locmoe_cos_hist(sh, x, idx, e, j, nb, lo, hi, he, hj, n)
    torch.cuda.synchronize()
    idx_h = idx.cpu().numpy()
    n_o, he_o, hj_o, ce, cj = P.oracle.cos_hist(W.host_bits(x), sh.x_dtype, w.E, idx_h, e, j, nb, lo, hi)
    assert n.item() == n_o == int((idx_h == e).sum()) and n_o > 0
    edges = lo + (hi - lo) * np.arange(nb + 1) / nb
    sel = idx_h == e
    for got, want, c in ((he, he_o, ce[sel]), (hj, hj_o, cj[sel])):
        got = got.cpu().numpy().astype(np.int64)
        assert got.sum() == n_o
        near = int((np.abs(c[:, None] - edges[None, :]).min(1) < 1e-6).sum())
        assert np.abs(got - want).sum() <= 2 * near
    # the routed cosines are the gate's own cos_sim output
    assert np.allclose(cs.cpu().numpy()[sel], ce[sel], rtol=1e-5, atol=1e-7)


def test_row_major_dispatch_without_slot(P):
    # locmoe_dispatch with slot = NULL (row-major kernels) writes the same buffer as the token-major call
    import torch
    B, W = P.B, P.W
    w = W.CONFIGS[2].scaled(3000)
    dev = torch.device("cuda:0")
    x, src = W.make_tokens(w, dev), W.make_src(w, dev)
    sh = B.make_shape(w.T, w.H, w.E, w.n_nodes, w.dev_per_node, x.dtype)
    Ca = B.conventional_capacity(w.T, sh.D, w.E, 1.0)
    st = B.make_router(sh, Ca, B.CapacityRule(1.0, 1.0, -1.0, 0, 0), dev)
    B.router_forward(st, x, src)
    torch.cuda.synchronize()
    want = st.buf.clone()
    assert int((st.inv < 0).sum()) > 0 and int((st.slot < 0).sum()) > 0   # empty rows and dropped tokens both occur
    st.buf.fill_(7.0)
    B.locmoe_dispatch(sh, Ca, x, st.inv, st.buf, True, None)
    torch.cuda.synchronize()
    assert torch.equal(st.buf.view(torch.int16), want.view(torch.int16))


def test_flat_dispatch_variant(P, monkeypatch):
    # the flat (row, vector) row-major kernel, forced although slot[] is supplied
    monkeypatch.setenv("LOCMOE_DISPATCH", "flat")
    P.run_staged(P.W.CONFIGS[2].scaled(6000), 1.25, full=True)
    P.run_staged(P.W.CONFIGS[1], 1.0, layout=1, full=True)


def test_plain_launches_without_programmatic_dependent_launch():
    # LOCMOE_PDL=0 is read once per process: run the staged comparison in a child process
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    code = ("import oracle; oracle.build(); from tests import parity as P; "
            "P.run_staged(P.W.CONFIGS[2].scaled(6000), 1.0, full=True); "
            "P.run_staged(P.W.CONFIGS[1], 1.0, layout=1, full=True, fused=False); print('ok')")
    env = dict(os.environ, LOCMOE_PDL="0")
    r = subprocess.run([sys.executable, "-c", code], cwd=root, env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and r.stdout.strip().endswith("ok"), r.stderr[-2000:]
