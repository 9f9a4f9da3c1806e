#!/usr/bin/env python
"""Benchmark of the LocMoE router hot path on B200: routed tokens/s and achieved HBM GB/s.

One "step" is one pass of the whole path -- gate, capacity, route, dispatch,
combine -- over one batch of T synthetic tokens.  Default workload: the
PanGu-Sigma-like layer (T = 65536, H = 5120, E = 64, bf16 tokens, 8 x 8 logical
devices, capacity factor 1.0).  With N > 1 (torchrun) every rank routes its own
batch on its own GPU (the path needs no exchange step on one logical-device
map), so the reported value is the aggregate and scaling is weak.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--cf F] [--impl reference]
                    [--variant router|peer8|topk2|peer] [--slices S] [--no-other-configs]

The timed region is exactly K replays of the step (a CUDA graph); per-stage times come from a separate
pass of eager steps with CUDA events between the stages (medians), the gate also launched on its own.
The default line (config 2) also carries short runs of the other configurations (`other_configs`).
`--variant peer` is the form with one rank per GPU and the exchange fused into dispatch and combine
(peer stores / loads; N = 1 works on one GPU).  `--impl reference` times the CPU oracle instead.

Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "routed tokens/sec (gate+dispatch+combine) and achieved HBM GB/s vs B200 peak, 1 GPU"
UNIT = "tokens/s"
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0     # the nominal HBM3e figure the 70 % target is stated against


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=400)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--config", type=int, default=2, help="workload 1..5 (default 2, the metric's configuration)")
    ap.add_argument("--cf", type=float, default=1.0,
                    help="capacity factor (both knobs); 0 = the literal-minimum mode: Theorem 1's minimum alone (multiplier 1)")
    ap.add_argument("--layout", choices=["send", "recv"], default="send")
    ap.add_argument("--impl", choices=["b200", "reference"], default="b200")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=48, help="end-to-end steps (the three-stream pipeline needs a few steps to fill)")
    ap.add_argument("--no-graph", action="store_true", help="launch every step eagerly instead of replaying a CUDA graph")
    ap.add_argument("--stage-steps", type=int, default=24,
                    help="eager steps with per-stage CUDA events after the timed region (median per stage; at least 20)")
    ap.add_argument("--other-steps", type=int, default=20, help="timed steps of each of the other configurations")
    ap.add_argument("--no-other-configs", action="store_true",
                    help="skip the short runs of configurations 1, 3, 4 and 5 that the default line carries")
    ap.add_argument("--variant", choices=["router", "peer8", "topk2", "peer"], default="router",
                    help="router: the metric's path; peer8: dispatch / combine through a table of eight receive buffers "
                         "(the fused-exchange kernels, all buffers on this GPU); topk2: the top-2 variant; peer: one rank "
                         "per GPU, each routing the tokens of its own logical source devices and storing them straight "
                         "into the receive buffers of the GPUs that host the experts (exchange.peer_layer_forward)")
    ap.add_argument("--fuse-gate", action="store_true",
                    help="gate, capacity and route as the one call locmoe_gate_route (the gate's time is then part of that stage)")
    ap.add_argument("--unfused", action="store_true", help="capacity and route as two calls instead of locmoe_capacity_route")
    ap.add_argument("--no-ffn", action="store_true", help="config 5 only: identity experts instead of the expert FFN")
    ap.add_argument("--ffn-inner", type=int, default=10240, help="config 5: inner size F of the expert FFN")
    ap.add_argument("--slices", type=int, default=1,
                    help="--variant peer with the expert FFN (config 5): expert blocks per rank, the exchange of block s+1 "
                         "overlapping the experts of block s")
    ap.add_argument("--tokens", type=int, default=0, help="override T (profiling-sized case; not the metric's workload)")
    return ap.parse_args()


def measured_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def measured_tensor_peak():
    """Sustained cuBLAS bf16 rate of this pool (the FFN runs inside a long step), else the fallback figure."""
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["bf16_tflops_sustained"]), "measured (cuBLAS bf16 sustained, MEASURED_PEAKS.json)"
    except Exception:
        return 1400.0, "fallback"


def measured_tensor_burst():
    """cuBLAS bf16 rate of a kernel timed alone (burst), for context beside the sustained figure."""
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["bf16_tflops"])
    except Exception:
        return 1590.0


class ClockSampler(threading.Thread):
    """Reads SM clock and throttle reasons through NVML while the timed region runs (read-only)."""

    def __init__(self, index: int, period_s: float = 0.02):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
            getattr(nv, "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80): "hw_power_brake",
        }
        while not self._stop_evt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop_evt.wait(self.period)

    def stop(self):
        self._stop_evt.set()
        if self.is_alive():
            self.join(timeout=2)
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2] if s else None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(s)}


def physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


def oracle_step(oracle, xh, srch, dtype_code, w, cf, layout):
    """One pass of the whole path in the CPU oracle on host arrays; returns kept tokens."""
    T = xh.shape[0]
    g = oracle.gate(xh, dtype_code, w.E)
    cap = oracle.capacity(g.idx, g.cos, w.E, w.H, w.D, min_mult=cf if cf > 0 else 1.0, capacity_factor=cf)
    C = cap.C_local
    r = oracle.route(g.idx, srch, w.E, w.n_nodes, w.dev_per_node, C, C, layout)
    rows = w.D * w.E * C
    buf = oracle.dispatch(xh, dtype_code, r.slot, rows)
    out = oracle.combine(buf, dtype_code, r.slot, g.R)
    return int((r.slot >= 0).sum()), out.shape


def run_reference(args):
    """The CPU oracle as the reference arm: same metric, bounded sample per step, host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy as np
    import oracle
    from paper_2401_13920_b200 import workloads as W
    oracle.build()
    w = W.CONFIGS[args.config]
    dtc = 0 if w.dtype == "f32" else 1
    layout = 0 if args.layout == "send" else 1
    # calibrate on a small sample, then size the per-step sample so that the run ends within ~2 minutes
    probe = w.scaled(min(w.T, 1024))
    xh = W.host_bits(W.make_tokens(probe, "cpu"))
    sh = W.make_src(probe, "cpu").numpy()
    t0 = time.perf_counter()
    oracle_step(oracle, xh, sh, dtc, probe, args.cf, layout)
    per_tok = (time.perf_counter() - t0) / probe.T
    total_steps = args.steps + args.warmup
    n = int(max(256, min(w.T, 120.0 / max(total_steps, 1) / per_tok)))
    n -= n % w.D if n >= w.D else 0
    sub = w.scaled(n)
    xh = W.host_bits(W.make_tokens(sub, "cpu"))
    sh = W.make_src(sub, "cpu").numpy()
    for _ in range(args.warmup):
        oracle_step(oracle, xh, sh, dtc, sub, args.cf, layout)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(oracle, xh, sh, dtc, sub, args.cf, layout)
    dt = time.perf_counter() - t0
    val = n * args.steps / dt
    sample = "first %d tokens of the workload per step, whole path, single thread, gcc -O2" % n
    line = {
        "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic", "impl": "reference",
        "config": workload_config(w, args), "sample_tokens_per_step": n,
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "host_cores": os.cpu_count(),
    }
    print(json.dumps(line))


def workload_config(w, args, n_tokens=None):
    return {
        "workload": "config %d (%s): T=%d H=%d E=%d %s tokens, %dx%d logical devices, c_f=%g, %s layout" % (
            w.config, w.name, n_tokens or w.T, w.H, w.E, w.dtype, w.n_nodes, w.dev_per_node, args.cf, args.layout),
        "expert_ffn": bool((w.config % 10) == 5 and not getattr(args, "no_ffn", False) and getattr(args, "variant", "router") == "router"),
        "variant": {"router": "the metric's path (top-1, one GPU)",
                    "peer8": "dispatch / combine through a table of eight receive buffers (fused-exchange kernels, all on this GPU)",
                    "topk2": "top-2 variant: 2T assignments routed, two-term combine",
                    "peer": "fused exchange: every rank routes its own source devices' tokens and stores them into the "
                            "owners' receive buffers (peer stores / loads; identity experts)"}[getattr(args, "variant", "router")],
        "T": n_tokens or w.T, "H": w.H, "E": w.E, "token_dtype": w.dtype, "n_nodes": w.n_nodes,
        "dev_per_node": w.dev_per_node, "capacity_factor": args.cf, "layout": args.layout,
        "l2": "inputs exceed the 126 MB L2, no flush" if (n_tokens or w.T) * w.H * (2 if w.dtype == "bf16" else 4) > 126e6
        else "inputs fit in L2 (latency-bound configuration)",
        "stands_in_for": "the paper's private corpus activations (not available); i.i.d. synthetic tokens",
    }


def median(v):
    s = sorted(v)
    n = len(s)
    return float(s[n // 2] if n % 2 else 0.5 * (s[n // 2 - 1] + s[n // 2]))


def measure(args, w, env, *, steps, warmup, stage_steps, use_ffn, variant, fuse_gate, fused, e2e_steps, cpu_baseline_s):
    """Builds the workload on the device, times K steps of the whole path (CUDA events on the launching stream,
    barrier + synchronize on both sides, max over ranks), then takes per-stage times from a separate pass of eager
    steps with events between the stages (median).  Returns the pieces of the JSON line."""
    import numpy as np
    import torch
    from paper_2401_13920_b200 import binding as B
    from paper_2401_13920_b200 import sharding
    from paper_2401_13920_b200 import workloads as W

    dev, dist, world, rank, local_rank = env["dev"], env["dist"], env["world"], env["rank"], env["local_rank"]
    if variant == "peer":
        return measure_peer(args, w, env, steps=steps, warmup=warmup, stage_steps=stage_steps)
    layout_name = args.layout
    if use_ffn or variant == "peer8":
        layout_name = "recv"      # the expert FFN and the peer kernels work on the receive-side layout
    layout = B.LAYOUT_SEND if layout_name == "send" else B.LAYOUT_RECV
    x = W.make_tokens(w, dev)
    src = W.make_src(w, dev)
    shape = B.make_shape(w.T, w.H, w.E, w.n_nodes, w.dev_per_node, x.dtype, layout)
    rule = B.CapacityRule(args.cf if args.cf > 0 else 1.0, args.cf, -1.0, B.BOUND_BETA, 0)   # c_f = 0: the minimum alone
    C_alloc = B.conventional_capacity(w.T, shape.D, w.E, args.cf)
    st = B.make_router(shape, C_alloc, rule, dev)
    y = None
    if w.y_dtype == "f32":
        y = W.make_expert_out(w, st.rows, dev, "f32")
    F = args.ffn_inner
    w_in = w_out = h1 = None
    if use_ffn:
        w_in, w_out = W.make_expert_weights(w, F, dev)
        h1 = torch.empty(st.rows, F, dtype=torch.bfloat16, device=dev)
        y = torch.empty(st.rows, w.H, dtype=torch.bfloat16, device=dev)
    ysrc = st.buf if y is None else y

    stream = torch.cuda.current_stream()
    stages = (["gate_route"] if fuse_gate else ["gate"] + (["capacity_route"] if fused else ["capacity", "route"])) + \
             ["dispatch"] + (["ffn"] if use_ffn else []) + ["combine"]

    tk = None
    if variant == "peer8":
        n_peers = 8
        while shape.D % n_peers:
            n_peers //= 2
        rpp = st.rows // n_peers
        peer_bufs = [st.buf[q * rpp:(q + 1) * rpp] for q in range(n_peers)]   # eight receive buffers, all on this GPU
        stages = ["gate", "capacity_route", "dispatch", "combine"]
    elif variant == "topk2":
        K2 = 2
        C_alloc = B.conventional_capacity(K2 * w.T, shape.D, w.E, args.cf)
        tk = B.make_topk_state(shape, K2, C_alloc, dev)
        src_k = src.repeat(K2).contiguous()
        stages = ["gate", "capacity", "select", "route", "dispatch", "combine"]

    def step(ev=None):
        sh, Ca = st.shape, st.C_alloc
        i = 0
        def mark():
            nonlocal i
            if ev:
                ev[i].record(stream)
            i += 1
        if variant == "topk2":
            B.topk_forward(tk, x, src_k, rule, stream=stream, mark=mark)
            return
        if variant == "peer8":
            mark()
            B.locmoe_gate(sh, x, None, st.idx, st.gate_w, st.cos_sim, None, stream)
            mark()
            B.locmoe_capacity_route(sh, st.idx, st.cos_sim, src, st.rule, st.delta_e, st.theta_e, st.cap_dev, Ca, st.pos,
                                    st.slot, st.drop, st.inv, st.counts, st.kept, st.send_counts, st.load, st.locality,
                                    st.status, st.ws, stream, early_init=not ev)
            mark()
            B.locmoe_dispatch_peer(sh, Ca, x, st.inv, st.slot, peer_bufs, 0, sh.D, True, stream)
            mark()
            B.locmoe_combine_peer(sh, Ca, peer_bufs, B.dtype_code(x.dtype), st.slot, st.gate_w, st.out, stream)
            mark()
            return
        mark()
        if fuse_gate:
            B.locmoe_gate_route(sh, x, None, src, st.rule, st, stream)
        else:
            B.locmoe_gate(sh, x, None, st.idx, st.gate_w, st.cos_sim, None, stream)
            mark()
        if fuse_gate:
            pass
        elif fused:
            B.locmoe_capacity_route(sh, st.idx, st.cos_sim, src, st.rule, st.delta_e, st.theta_e, st.cap_dev, Ca, st.pos,
                                    st.slot, st.drop, st.inv, st.counts, st.kept, st.send_counts, st.load, st.locality,
                                    st.status, st.ws, stream, early_init=not ev)   # eager steps record an event in between
        else:
            B.locmoe_capacity(sh, st.idx, st.cos_sim, st.rule, st.delta_e, st.theta_e, st.cap_dev, st.ws, stream)
            mark()
            B.locmoe_route(sh, st.idx, src, st.cap_dev, Ca, st.pos, st.slot, st.drop, st.inv, st.counts, st.kept,
                           st.send_counts, st.load, st.locality, st.status, st.ws, stream)
        mark()
        B.locmoe_dispatch(sh, Ca, x, st.inv, st.buf, True, stream, slot=st.slot)
        mark()
        if use_ffn:
            B.locmoe_expert_ffn(sh, Ca, F, st.buf, w_in, w_out, h1, y, stream)
            mark()
        B.locmoe_combine(sh, Ca, ysrc, st.slot, st.gate_w, st.out, False, stream)
        mark()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    warmup = max(warmup, 3)
    for _ in range(warmup):
        step()
    barrier()

    # ---- timed region: exactly K steps, device-timed; the step is captured once in a CUDA graph and replayed ----
    K = steps
    graph = None
    if not args.no_graph:
        side = torch.cuda.Stream(dev)
        side.wait_stream(stream)
        with torch.cuda.stream(side):
            stream_backup = stream
            stream = side
            step()                     # one eager pass on the capture stream (lazy initialisation outside capture)
            side.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                step()
            stream = stream_backup
        torch.cuda.current_stream().wait_stream(side)
        graph.replay()
    sampler = ClockSampler(physical_gpu_index(local_rank), period_s=0.001)
    sampler.start()
    barrier()
    t_start = torch.cuda.Event(enable_timing=True)
    t_end = torch.cuda.Event(enable_timing=True)
    t_start.record(stream)
    for k in range(K):
        if graph is None:
            step()
        else:
            graph.replay()
    t_end.record(stream)
    barrier()
    n_timed = len(sampler.samples)
    total_ms = sharding.max_over_ranks(t_start.elapsed_time(t_end), dev)
    ms_per_step = total_ms / K
    value = world * w.T * K / (total_ms * 1e-3)

    # ---- per-stage times: a separate pass of eager steps with CUDA events between the stages on the launching
    #      stream (an event record costs ~2.5 us of stream time, so the timed region above carries none); medians ----
    S = max(int(stage_steps), 20)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(len(stages) + 1)] for _ in range(S)]
    for k in range(S):
        step(evs[k])
    barrier()
    # the gate kernel launched back to back on its own (no other kernel's dirty lines to write back under it)
    gate_alone_ms = None
    if variant == "router" and not fuse_gate:
        ga = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(S)]
        for k in range(S):
            ga[k][0].record(stream)
            B.locmoe_gate(st.shape, x, None, st.idx, st.gate_w, st.cos_sim, None, stream)
            ga[k][1].record(stream)
        barrier()
        gate_alone_ms = median([g[0].elapsed_time(g[1]) for g in ga])
    clocks = sampler.stop()
    clocks["samples_in_timed_region"] = n_timed
    clocks["covers"] = "timed region and per-stage pass"
    stage_ms = {s: median([evs[k][i].elapsed_time(evs[k][i + 1]) for k in range(S)]) for i, s in enumerate(stages)}
    flags = B.locmoe_device_flags()
    if flags != 0:
        raise RuntimeError("a kernel gave up a bounded wait during the bench (device flags %d): the timing is void" % flags)

    # ---- algorithmic bytes per launch (per token: see the per-kernel byte model in the design notes) ----
    slot_t = tk["slot"] if tk is not None else st.slot
    kept = int((slot_t >= 0).sum().item())            # kept assignments (tokens, or token-choice pairs for top-k)
    bx = x.element_size()
    by = ysrc.element_size()
    rows = st.rows if tk is None else shape.D * w.E * C_alloc
    bytes_per_launch = {
        "gate": w.T * w.H * bx + 12 * w.T + (4 * w.T * w.E if tk is not None else 0),
        "dispatch": kept * w.H * bx + rows * w.H * bx + 4 * rows,
        "combine": kept * w.H * by + w.T * w.H * bx + 8 * w.T * (tk["K"] if tk is not None else 1),
    }
    peak, peak_kind = measured_peak()
    if fuse_gate:   # the gate's bytes over the time of the whole gate + capacity + route chain
        bytes_per_launch = {"gate_route": bytes_per_launch["gate"], "dispatch": bytes_per_launch["dispatch"],
                            "combine": bytes_per_launch["combine"]}
    hbm_stages = tuple(bytes_per_launch)
    kernels = {}
    for s in hbm_stages:
        gbs = bytes_per_launch[s] / (stage_ms[s] * 1e-3) / 1e9
        kernels[s] = {"ms": stage_ms[s], "bytes": bytes_per_launch[s], "achieved_gbs": gbs, "frac": gbs / peak,
                      "frac_nominal": gbs / NOMINAL_HBM_GBS}
    if gate_alone_ms is not None:
        g = bytes_per_launch["gate"] / (gate_alone_ms * 1e-3) / 1e9
        kernels["gate"].update({"alone_ms": gate_alone_ms, "alone_gbs": g, "alone_frac": g / peak, "alone_frac_nominal": g / NOMINAL_HBM_GBS,
                                "note": "ms / frac: inside the step, where the previous kernel's last ~55 MB of output are still dirty "
                                        "in L2 and are written back under this kernel; alone_*: the same launch repeated back to back"})
    dominant = max(hbm_stages, key=lambda s: stage_ms[s])
    traffic = ncu_traffic(dominant, w, args.cf, args.tokens) if variant == "router" else None
    path_bytes = sum(bytes_per_launch.values())
    path_gbs = path_bytes / (ms_per_step * 1e-3) / 1e9
    if use_ffn:     # the router path's bytes over the time of its own stages (the tensor-bound stage left out)
        hbm_ms = sum(v for k, v in stage_ms.items() if k != "ffn")
        path_gbs = path_bytes / (hbm_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": dominant, "achieved": kernels[dominant]["achieved_gbs"], "peak": peak,
                "peak_kind": peak_kind + " (copy, MEASURED_PEAKS.json)" if peak_kind == "measured" else "fallback",
                "unit": "GB/s", "frac": kernels[dominant]["frac"], "frac_nominal": kernels[dominant]["frac_nominal"],
                "nominal_peak": NOMINAL_HBM_GBS, "traffic": traffic,
                "traffic_source": None if traffic is None else
                "ncu capture of this workload and launch configuration summarised in profiles/dram_traffic_config2.md; "
                "not measured in this run",
                "path_bytes": path_bytes, "path_frac": path_gbs / peak, "path_frac_nominal": path_gbs / NOMINAL_HBM_GBS,
                "kernels": kernels, "stage_ms": stage_ms,
                "stage_ms_how": "median of %d eager steps after the timed region, CUDA events between the stages" % S}
    if use_ffn:
        # the expert FFN dominates: two grouped GEMMs, 2 * 2 * rows * H * F flops, tensor-core bound
        flops = 4.0 * rows * w.H * F
        tf = flops / (stage_ms["ffn"] * 1e-3) / 1e12
        tpeak, tkind = measured_tensor_peak()
        roofline.update({"bound": "tensor", "kernel": " + ".join(B.FFN_KERNEL_NAMES[k] for k in B.locmoe_ffn_kernels(st.shape, st.C_alloc, F)) + " (the library's choice per GEMM)", "achieved": tf, "peak": tpeak,
                         "peak_kind": tkind, "unit": "TFLOP/s", "frac": tf / tpeak, "traffic": None, "traffic_source": None,
                         "flops": flops, "frac_of_burst_peak": tf / measured_tensor_burst(), "hbm_kernels": kernels})
        roofline.pop("frac_nominal", None)

    launches = B.locmoe_launch_counts(shape)
    if variant == "topk2":
        lv = B.locmoe_launch_counts(tk["shape_v"])
        launches = {"gate": 1, "capacity": launches["capacity"], "select": 1, "route": lv["route"] + 1, "dispatch": 1, "combine": 1}
    elif fuse_gate:
        launches = {"gate_route": launches["route"], "dispatch": launches["dispatch"], "combine": launches["combine"]}
    elif fused:
        # the capacity stage rides on the route stage's launches (up to 8192 experts)
        cr = launches.pop("route") + (launches["capacity"] if shape.E > 8192 else 0)
        launches.pop("capacity")
        launches = {"gate": launches["gate"], "capacity_route": cr, "dispatch": launches["dispatch"], "combine": launches["combine"]}
    if use_ffn:
        launches["ffn"] = 2
    cap = B.locmoe_capacity_read(tk["cap_dev"] if tk is not None else st.cap_dev)

    # ---- end to end: host buffers in, host buffers out, copies inside the timed region ----
    e2e = None
    if e2e_steps > 0 and not use_ffn and variant == "router":
        xh = torch.empty(x.shape, dtype=x.dtype, pin_memory=True)
        xh.copy_(x)
        srch = torch.empty(src.shape, dtype=src.dtype, pin_memory=True)
        srch.copy_(src)
        outh = [torch.empty(st.out.shape, dtype=st.out.dtype, pin_memory=True) for _ in range(2)]
        hr = B.HostRouter(shape, C_alloc, rule, dev)
        for i in range(3):
            hr.forward(xh, srch, outh[i & 1], y=y)
        hr.synchronize()
        barrier()
        a = torch.cuda.Event(enable_timing=True)
        b = torch.cuda.Event(enable_timing=True)
        a.record(hr.s_in)
        for i in range(e2e_steps):
            hr.forward(xh, srch, outh[i & 1], y=y)
        hr.s_out.wait_stream(hr.s_comp)
        hr.s_out.wait_stream(hr.s_in)
        b.record(hr.s_out)
        hr.synchronize()
        barrier()
        ems = sharding.max_over_ranks(a.elapsed_time(b), dev)
        e2e = {"value": world * w.T * e2e_steps / (ems * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": xh.numel() * xh.element_size() + srch.numel() * 4,
               "d2h_bytes_per_step": outh[0].numel() * outh[0].element_size(), "steps": e2e_steps,
               "api": "binding.HostRouter.forward on pinned host tensors (copy in, five C-ABI calls, copy out; "
                      "successive steps pipelined over three streams)"}
        del hr, xh, outh

    # ---- CPU baseline: the oracle, as it stands, on the host cores (rank 0, N = 1 only) ----
    cpu_baseline = None
    if rank == 0 and world == 1 and cpu_baseline_s > 0:
        import oracle
        oracle.build()
        n = min(w.T, 65536)
        xs = W.host_bits(x[:n])
        ss = src[:n].cpu().numpy()
        sub = w.scaled(n)
        reps, t0 = 0, time.perf_counter()
        while True:
            oracle_step(oracle, xs, ss, shape.x_dtype, sub, args.cf, layout)
            reps += 1
            dt = time.perf_counter() - t0
            if dt >= cpu_baseline_s or reps >= 64:
                break
        cpu_baseline = {"value": n * reps / dt, "unit": UNIT, "cores": 1, "kind": "oracle", "seconds": dt,
                        "sample": "first %d tokens of the workload, whole path %d times, single thread, gcc -O2 "
                                  "(host has %d cores)" % (n, reps, os.cpu_count())}

    args_l = argparse.Namespace(**{**vars(args), "layout": layout_name, "no_ffn": not use_ffn, "variant": variant})
    return {
        "value": value, "ms_per_step": ms_per_step, "steps": K, "warmup": warmup, "config": workload_config(w, args_l),
        "clocks": clocks, "e2e": e2e, "launches": launches, "graph": graph is not None,
        "roofline": roofline, "cpu_baseline": cpu_baseline,
        "routing": {"kept_fraction": kept / w.T, "C_local": cap.C_local, "C_expert": cap.C_expert, "delta": cap.delta,
                    "ec_min": cap.ec_min, "rows": rows, "kept_tokens_per_s": value * kept / w.T},
    }


def measure_peer(args, w, env, *, steps, warmup, stage_steps):
    """The fused exchange at N ranks: rank r owns the logical devices [r D/N, (r+1) D/N) and draws w.T tokens that
    come from them (weak scaling: N * w.T tokens in the whole batch, the capacity rule counts all of them); every
    rank routes its tokens in the receive-side layout of the whole map, stores kept rows into the owners' buffers
    (peer stores), and combines through peer loads; identity experts.  The host orders the steps across ranks
    (barriers inside exchange.peer_layer_forward), so the step is launched eagerly, not as a CUDA graph."""
    import torch
    from paper_2401_13920_b200 import binding as B
    from paper_2401_13920_b200 import exchange, sharding
    from paper_2401_13920_b200 import workloads as W

    dev, dist, world, rank, local_rank = env["dev"], env["dist"], env["world"], env["rank"], env["local_rank"]
    D = w.n_nodes * w.dev_per_node
    devs = sharding.devices_of_rank(D, world, rank)
    x = W.make_tokens(w, dev)                                       # this rank's tokens (its own seed when N > 1)
    src = (devs.start + torch.arange(w.T, device=dev, dtype=torch.int64) % len(devs)).to(torch.int32)
    T_global = world * w.T
    shape = B.make_shape(w.T, w.H, w.E, w.n_nodes, w.dev_per_node, x.dtype, B.LAYOUT_RECV)
    rule = B.CapacityRule(args.cf, args.cf, -1.0, B.BOUND_BETA, 0)
    C_alloc = B.conventional_capacity(T_global, D, w.E, args.cf)
    rows = D * w.E * C_alloc
    st = B.make_router(shape, C_alloc, rule, dev, with_buffer=False)
    recv = exchange.PeerBuffers(rows // world, w.H, x.dtype, dev)   # this rank's slice of the receive buffer
    stream = torch.cuda.current_stream()
    stages = ["gate", "capacity_route", "dispatch_peer", "experts", "combine_peer"]
    use_ffn = (w.config % 10) == 5 and not args.no_ffn
    F = args.ffn_inner
    y, w_in, w_out, h1, ffn_stream = recv, None, None, None, None
    if use_ffn:                                                     # this rank's experts: E / world of them
        w_all_in, w_all_out = W.make_expert_weights(w, F, dev)
        El = w.E // world
        w_in, w_out = w_all_in[rank * El:(rank + 1) * El].contiguous(), w_all_out[rank * El:(rank + 1) * El].contiguous()
        del w_all_in, w_all_out
        y = exchange.PeerBuffers(rows // world, w.H, torch.bfloat16, dev)
        h1 = torch.empty(rows // world, F, dtype=torch.bfloat16, device=dev)
        ffn_stream = torch.cuda.Stream(dev) if args.slices > 1 else None

    def step(ev=None):
        i = 0
        def mark():
            nonlocal i
            if ev:
                ev[i].record(stream)
            i += 1
        exchange.peer_layer_forward(B, sharding, shape, C_alloc, rule, x, src, recv, y, st, w_in, w_out, F, h1, stream=stream,
                                    mark=mark, slices=args.slices if use_ffn else 1, ffn_stream=ffn_stream)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    warmup = max(warmup, 3)
    for _ in range(warmup):
        step()
    barrier()
    sampler = ClockSampler(physical_gpu_index(local_rank), period_s=0.001)
    sampler.start()
    barrier()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record(stream)
    for _ in range(steps):
        step()
    t1.record(stream)
    barrier()
    n_timed = len(sampler.samples)
    total_ms = sharding.max_over_ranks(t0.elapsed_time(t1), dev)
    S = max(int(stage_steps), 20)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(len(stages) + 1)] for _ in range(S)]
    for k in range(S):
        step(evs[k])
    barrier()
    clocks = sampler.stop()
    clocks["samples_in_timed_region"] = n_timed
    stage_ms = {s: median([evs[k][i].elapsed_time(evs[k][i + 1]) for k in range(S)]) for i, s in enumerate(stages)}
    if B.locmoe_device_flags() != 0:
        raise RuntimeError("a kernel gave up a bounded wait during the bench")
    kept = int((st.slot >= 0).sum().item())
    sc = st.send_counts.view(D, D)[devs.start:devs.stop]           # kept rows of my sources per destination device
    own = int(sc[:, devs.start:devs.stop].sum().item())
    to_peers = (int(sc.sum().item()) - own) * w.H * x.element_size()
    bx = x.element_size()
    rows_mine = rows // world                                      # rows this rank zero-fills / owns on average
    bytes_per_launch = {"gate": w.T * w.H * bx + 12 * w.T,
                        "dispatch_peer": kept * w.H * bx + rows_mine * w.H * bx + 4 * rows_mine,
                        "combine_peer": kept * w.H * bx + w.T * w.H * bx + 8 * w.T}
    peak, peak_kind = measured_peak()
    kernels = {}
    for s_, b_ in bytes_per_launch.items():
        gbs = b_ / (stage_ms[s_] * 1e-3) / 1e9
        kernels[s_] = {"ms": stage_ms[s_], "bytes": b_, "achieved_gbs": gbs, "frac": gbs / peak, "frac_nominal": gbs / NOMINAL_HBM_GBS}
    ms_per_step = total_ms / steps
    path_bytes = sum(bytes_per_launch.values())
    path_gbs = path_bytes / (ms_per_step * 1e-3) / 1e9
    dominant = max(bytes_per_launch, key=lambda s_: stage_ms[s_])
    link_gbs = to_peers / (stage_ms["dispatch_peer"] * 1e-3) / 1e9 if to_peers else 0.0
    roofline = {"bound": "hbm" if world == 1 else "hbm / nvlink", "kernel": dominant, "achieved": kernels[dominant]["achieved_gbs"],
                "peak": peak, "peak_kind": peak_kind + " (copy, MEASURED_PEAKS.json)" if peak_kind == "measured" else "fallback",
                "unit": "GB/s", "frac": kernels[dominant]["frac"], "frac_nominal": kernels[dominant]["frac_nominal"],
                "nominal_peak": NOMINAL_HBM_GBS, "traffic": None, "traffic_source": None, "path_bytes": path_bytes,
                "path_frac": path_gbs / peak, "path_frac_nominal": path_gbs / NOMINAL_HBM_GBS, "kernels": kernels,
                "stage_ms": stage_ms, "stage_ms_how": "median of %d eager steps, CUDA events between the stages" % S,
                "peer": {"world": world, "bytes_to_peers_per_step": to_peers, "bytes_from_peers_per_step": to_peers,
                         "peer_store_gbs_per_rank": link_gbs, "nvlink_measured_gbs_per_direction": 770.0,
                         "expert_ffn": use_ffn, "slices": args.slices if use_ffn else 1,
                         "note": "stage times of dispatch_peer / experts include the host-ordered barrier across ranks; with "
                                 "slices > 1 dispatch_peer is the main stream's share (the windowed stores) and experts the wait "
                                 "for the second stream"}}
    cap = B.locmoe_capacity_read(st.cap_dev)
    launches = B.locmoe_launch_counts(shape)
    launches = {"gate": 1, "capacity": launches["capacity"], "capacity_route": launches["route"], "dispatch_peer": 1, "combine_peer": 1}
    args_l = argparse.Namespace(**{**vars(args), "layout": "recv", "no_ffn": True, "variant": "peer"})
    cfg = workload_config(w, args_l)
    cfg["T_global"] = T_global
    cfg["expert_ffn"] = use_ffn
    return {"value": world * w.T * steps / (total_ms * 1e-3), "ms_per_step": ms_per_step, "steps": steps, "warmup": warmup,
            "config": cfg, "clocks": clocks, "e2e": None, "launches": launches, "graph": False, "roofline": roofline,
            "cpu_baseline": None,
            "routing": {"kept_fraction": kept / w.T, "C_local": cap.C_local, "C_expert": cap.C_expert, "delta": cap.delta,
                        "ec_min": cap.ec_min, "rows": rows, "kept_tokens_per_s": world * kept * steps / (total_ms * 1e-3)}}


def summary_of(m):
    """Short record of one configuration for the `other_configs` object of the JSON line."""
    r = m["roofline"]
    ks = r.get("hbm_kernels", r["kernels"])
    out = {
        "workload": m["config"]["workload"], "expert_ffn": m["config"]["expert_ffn"], "steps": m["steps"], "warmup": m["warmup"],
        "ms_per_step": m["ms_per_step"], "tokens_per_s": m["value"],
        "kernels": {k: {kk: vv for kk, vv in v.items() if kk not in ("bytes", "note")} for k, v in ks.items()},
        "stage_ms": r["stage_ms"], "path_frac": r["path_frac"], "path_frac_nominal": r["path_frac_nominal"],
        "kept_fraction": m["routing"]["kept_fraction"], "C_local": m["routing"]["C_local"],
        "clocks": {k: m["clocks"][k] for k in ("sm_mhz", "sm_max_mhz", "reasons", "samples")},
        "launches_per_step": sum(m["launches"].values()),
    }
    if m["config"]["expert_ffn"]:
        out["ffn"] = {"ms": r["stage_ms"]["ffn"], "tflops": r["achieved"], "frac_of_sustained_peak": r["frac"],
                      "frac_of_burst_peak": r["frac_of_burst_peak"], "peak_sustained": r["peak"]}
    return out


def main():
    args = parse_args()
    if args.impl == "reference":
        return run_reference(args)

    import gc
    import torch
    from paper_2401_13920_b200 import binding as B   # raises if the CUDA library cannot be built / loaded
    from paper_2401_13920_b200 import workloads as W

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU path")
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)
    env = {"dev": dev, "dist": dist, "world": world, "rank": rank, "local_rank": local_rank}

    def workload(cfg, tokens=0):
        w = W.CONFIGS[cfg]
        if tokens > 0:
            w = w.scaled(tokens)
        if world > 1:
            # every rank routes its own batch: same shape, its own seed
            w = W.Workload(**{**w.__dict__, "config": w.config + 10 * rank, "name": w.name})
        return w

    w = workload(args.config, args.tokens)
    variant = args.variant
    use_ffn = (w.config % 10) == 5 and not args.no_ffn and variant == "router"
    m = measure(args, w, env, steps=args.steps, warmup=args.warmup, stage_steps=args.stage_steps, use_ffn=use_ffn,
                variant=variant, fuse_gate=args.fuse_gate and variant == "router", fused=not args.unfused,
                e2e_steps=args.e2e_steps, cpu_baseline_s=0.0 if args.no_cpu_baseline else 10.0)

    # ---- the other configurations, each a short run of the same bench (one GPU only; the headline stays above) ----
    others = None
    default_headline = args.config == 2 and args.tokens == 0 and variant == "router" and not args.fuse_gate and not args.unfused
    if world == 1 and default_headline and not args.no_other_configs:
        others = {}
        # the light configurations first, the power-hungry ones (config 4's 10 ms steps, the FFN) last, and a pause
        # before each so that none inherits the clocks the power cap left its predecessor with
        for name, cfg, ffn, cf in (("config1", 1, False, args.cf), ("config1_literal_minimum_capacity", 1, False, 0.0),
                                   ("config5_router_only", 5, False, args.cf),
                                   ("config5_literal_minimum_capacity", 5, False, 0.0),
                                   ("config2_literal_minimum_capacity", 2, False, 0.0), ("config3", 3, False, args.cf),
                                   ("config3_literal_minimum_capacity", 3, False, 0.0),
                                   ("config4_literal_minimum_capacity", 4, False, 0.0),
                                   ("config4", 4, False, args.cf), ("config5_with_ffn", 5, True, args.cf)):
            gc.collect()
            torch.cuda.empty_cache()
            time.sleep(1.0)
            try:
                args_o = argparse.Namespace(**{**vars(args), "cf": cf})
                mo = measure(args_o, workload(cfg), env, steps=args.other_steps, warmup=5, stage_steps=args.stage_steps,
                             use_ffn=ffn, variant="router", fuse_gate=False, fused=True, e2e_steps=0, cpu_baseline_s=0.0)
                others[name] = summary_of(mo)
                del mo
            except Exception as exc:   # a configuration that cannot run here is reported, the headline is kept
                others[name] = {"error": "%s: %s" % (type(exc).__name__, exc)}

    if rank == 0:
        line = {
            "metric": METRIC, "value": m["value"], "unit": UNIT, "n_gpus": world, "steps": m["steps"], "warmup": m["warmup"],
            "ms_per_step": m["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic", "config": m["config"],
            "clocks": m["clocks"], "e2e": m["e2e"], "gpu_launches": sum(m["launches"].values()) * m["steps"],
            "launches_per_step": m["launches"],
            "launch_mode": "CUDA graph replay of the step in the timed region; per-stage times from a separate eager pass"
                           if m["graph"] else "eager",
            "roofline": m["roofline"], "cpu_baseline": m["cpu_baseline"], "routing": m["routing"],
            "other_configs": others,
            "context": "the paper reports a 12.68%-22.24% per-epoch training-time reduction on 64-256 Ascend 910A NPUs; "
                       "it gives no number for this path",
        }
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu capture summarised in
# profiles/dram_traffic_config2.md, taken at the bench's full size.
NCU_TRAFFIC = {
    (2, 1.0): {"gate": 671117568 + 3323136, "dispatch": 606188288 + 612412416, "combine": 606180864 + 610791680},
}


def ncu_traffic(kernel: str, w, cf: float, tokens_override: int):
    if tokens_override:
        return None
    return NCU_TRAFFIC.get((w.config % 10, cf), {}).get(kernel)


if __name__ == "__main__":
    main()
