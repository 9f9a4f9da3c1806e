"""Two CPU ranks over gloo run `exchange.peer_layer_forward` with a recording stand-in for the binding and plain
tensors for the peer buffers: what is checked is the call SEQUENCE of one rank's layer pass with the exchange fused
into dispatch and combine -- barriers in the right places, the same batch-wide capacity rule on both ranks, the
peer tables and source-device ranges handed to the kernels -- which needs no GPU."""
import os
import socket
import sys

import pytest
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


class _Rule:
    def __init__(self, min_mult, capacity_factor, delta_override, bound_form, T_global):
        self.min_mult, self.capacity_factor, self.delta_override = min_mult, capacity_factor, delta_override
        self.bound_form, self.T_global = bound_form, T_global


class _Shape:
    def __init__(self, T, H, E, N, Dn, dt, layout):
        self.T, self.H, self.E, self.n_nodes, self.dev_per_node, self.x_dtype, self.layout = T, H, E, N, Dn, dt, layout
        self.D = N * Dn


class _RecordingBinding:
    """Stands in for `binding`: every kernel call is appended to `log`; the capacity call writes this rank's
    per-expert minima so that the host-side reduction has something to reduce."""
    LAYOUT_RECV = 1
    CapacityRule = _Rule

    def __init__(self, log, rank):
        self.log, self.rank = log, rank

    def make_shape(self, T, H, E, N, Dn, dt, layout):
        return _Shape(T, H, E, N, Dn, dt, layout)

    def dtype_code(self, dt):
        return 1

    def locmoe_gate(self, sh, x, eps, idx, gate_w, cos_sim, probs, stream):
        self.log.append(("gate", sh.T))

    def locmoe_capacity(self, sh, idx, cos_sim, rule, delta_e, theta_e, cap_dev, ws, stream):
        delta_e.copy_(torch.tensor([0.5, 0.25, 1.0, 0.75]) if self.rank == 0 else torch.tensor([0.125, 0.5, 1.0, -0.25]))
        self.log.append(("capacity", rule.delta_override, rule.T_global))

    def locmoe_capacity_route(self, sh, idx, cos_sim, src, rule, *rest):
        self.log.append(("capacity_route", rule.delta_override, rule.T_global, rule.min_mult, rule.capacity_factor))

    def locmoe_dispatch_peer(self, sh, C_alloc, x, inv, slot, pointers, lo, hi, zero_pad, stream, window=None):
        self.log.append(("dispatch_peer", tuple(pointers), lo, hi) + ((window,) if window is not None else ()))

    def locmoe_expert_ffn(self, sh, C, F, buf, w_in, w_out, h1, y, stream):
        self.log.append(("expert_ffn", sh.E, sh.n_nodes, sh.dev_per_node, C, F) + ((stream,) if stream is not None else ()))

    def locmoe_combine_peer(self, sh, C_alloc, pointers, ydt, slot, gate_w, out, stream):
        self.log.append(("combine_peer", tuple(pointers)))


class _PlainPeerBuffers:
    """The multi-rank branch of PeerBuffers without symmetric memory: a local tensor, made-up peer addresses, and a
    barrier that is logged and really is a barrier over the process group."""

    def __init__(self, name, rank, world, log):
        import torch.distributed as dist
        self.dist, self.name, self.world, self.log = dist, name, world, log
        self.local = torch.zeros(8, 4)
        self.pointers = [1000 * (q + 1) + (0 if name == "recv" else 7) for q in range(world)]

    def synchronize(self, stream=None):
        self.log.append(("synchronize", self.name))

    def barrier(self, stream=None):
        self.log.append(("barrier", self.name) + ((stream,) if stream is not None else ()))
        self.dist.barrier()

    def order(self, first, then):
        self.log.append(("order", first, then))


class _State:
    def __init__(self):
        self.idx = self.gate_w = self.cos_sim = self.theta_e = self.cap_dev = self.ws = None
        self.pos = self.slot = self.drop = self.inv = self.counts = self.kept = self.send_counts = None
        self.load = self.locality = self.status = None
        self.delta_e = torch.ones(4)
        self.out = torch.zeros(1)


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    from paper_2401_13920_b200 import exchange, sharding
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        log = []
        B = _RecordingBinding(log, rank)
        shape = _Shape(100 + 50 * rank, 64, 4, 2, 2, 1, 1)     # the ranks hold different numbers of tokens
        rule = _Rule(1.0, 1.25, -1.0, 0, 0)
        recv = _PlainPeerBuffers("recv", rank, world, log)
        y = _PlainPeerBuffers("y", rank, world, log)
        # pass 1: real experts, separate output buffers; pass 2: identity experts, y is recv
        exchange.peer_layer_forward(B, sharding, shape, 9, rule, None, None, recv, y, _State(), w_in=object(), w_out=object(),
                                    F=32, h1=None, stream=None)
        n1 = len(log)
        exchange.peer_layer_forward(B, sharding, shape, 9, rule, None, None, recv, recv, _State(), stream=None)
        n2 = len(log)
        # pass 3: the exchange overlapped with the experts, two blocks of one expert each
        exchange.peer_layer_forward(B, sharding, shape, 9, rule, None, None, recv, y, _State(), w_in=[0, 1], w_out=[0, 1],
                                    F=32, h1=torch.zeros(72, 32), stream="main", slices=2, ffn_stream="side")
        q.put((rank, log[:n1], log[n1:n2], log[n2:]))
    finally:
        dist.destroy_process_group()


def test_peer_layer_forward_call_sequence_on_two_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
    for rank, first, second, third in res:
        names = [c[0] for c in first]
        assert names[2] == "synchronize"                           # the stream is waited for before the minima are reduced
        first, names = first[:2] + first[3:], names[:2] + names[3:]
        assert names == ["gate", "capacity", "capacity_route", "dispatch_peer", "barrier", "expert_ffn", "barrier",
                         "combine_peer"], names
        assert first[0] == ("gate", 100 + 50 * rank)
        assert first[1] == ("capacity", -1.0, 0)                   # the rank's own minima are measured first
        # batch-wide rule: minimum over ranks and experts is -0.25, clamped to 0 (never "< 0 = measure"); 250 tokens
        assert first[2] == ("capacity_route", 0.0, 250, 1.0, 1.25)
        assert first[3] == ("dispatch_peer", (1000, 2000), 2 * rank, 2 * rank + 2)     # peer table, own source devices
        assert first[4] == ("barrier", "recv") and first[6] == ("barrier", "y")
        assert first[5] == ("expert_ffn", 2, 1, 1, 4 * 9, 32)       # this rank's two experts, D * C_alloc rows each
        assert first[7] == ("combine_peer", (1007, 2007))
        # identity experts in the receive buffer itself: no FFN call, and a trailing barrier after the combine
        second = second[:2] + second[3:]
        assert [c[0] for c in second] == ["gate", "capacity", "capacity_route", "dispatch_peer", "barrier", "barrier",
                                           "combine_peer", "barrier"]
        assert second[6] == ("combine_peer", (1000, 2000))
        # sliced pass: per block -- windowed peer stores, barrier on the main stream, stream order, that block's experts on
        # the side stream -- then the barrier on the side stream, the order back, the combine
        third = third[:2] + third[3:]
        assert [c[0] for c in third] == ["gate", "capacity", "capacity_route", "dispatch_peer", "barrier", "order", "expert_ffn",
                                          "dispatch_peer", "barrier", "order", "expert_ffn", "barrier", "order", "combine_peer"]
        assert third[3][4] == (0, 36) and third[7][4] == (36, 72)        # rows of block s inside every rank's slice
        assert third[4] == ("barrier", "recv", "main") and third[5] == ("order", "main", "side")
        assert third[6] == ("expert_ffn", 1, 1, 1, 36, 32, "side") and third[10][-1] == "side"
        assert third[11] == ("barrier", "y", "side") and third[12] == ("order", "side", "main")
    assert res[0][1][3] == res[1][1][3] and res[0][1][3][0] == "capacity_route"   # the same rule on both ranks
