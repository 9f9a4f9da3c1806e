"""The All-to-All around the experts (Sec. 3.2.4), as plain collectives: send-side buffer -> receive-side buffer.

`locmoe_route` / `locmoe_dispatch` fill a buffer whose rows are grouped by (source device, destination in
"self, own node, other nodes" order); the expert FFN wants the receive-side grouping (expert, source).  On one GPU
both are just layouts.  With one process per GPU, each owning a contiguous block of the logical devices, this module
moves the rows between the two layouts with ONE equal-split ``all_to_all_single`` per direction (NCCL over
NVLink/NVSwitch on GPUs, gloo on CPU in the tests).  Only integer permutations of fixed-size cells (C_alloc rows)
happen here; no router arithmetic.  This is the library-collective baseline for the exchange step, not a fused
compute+communication kernel.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


class ExchangePlan:
    """Cell permutations for one rank.  A cell is the block of C_alloc rows of one (source device, expert) pair."""

    def __init__(self, n_nodes: int, dev_per_node: int, E: int, world: int, rank: int):
        D = n_nodes * dev_per_node
        if D % world or E % D:
            raise ValueError("devices must divide over ranks and experts over devices")
        per, Ed = D // world, E // D
        a0 = rank * per
        self.D, self.Ed, self.per, self.world, self.rank = D, Ed, per, world, rank
        self.cells_local = per * D * Ed            # cells of this rank in either layout
        from . import binding
        r = lambda a, b: binding.dest_order(n_nodes, dev_per_node, a, b)   # the layout's r(a, b), from the library
        # send order: destination rank q, then source device a (mine), then destination device b (q's), then local expert
        send = []
        for q in range(world):
            for a in range(a0, a0 + per):
                for b in range(q * per, (q + 1) * per):
                    for el in range(Ed):
                        send.append(((a - a0) * D + r(a, b)) * Ed + el)          # SEND cell ((a, r(a,b)), el), local to me
        # what arrives: source rank p, then source device a (p's), then destination device b (mine), then local expert;
        # it belongs at RECV cell ((b, el), r(b, a)), local to me
        recv = []
        for p in range(world):
            for a in range(p * per, (p + 1) * per):
                for b in range(a0, a0 + per):
                    for el in range(Ed):
                        recv.append(((b - a0) * Ed + el) * D + r(b, a))
        self.send_cells = torch.tensor(send, dtype=torch.int64)
        self.recv_cells = torch.tensor(recv, dtype=torch.int64)
        assert sorted(send) == list(range(self.cells_local)) and sorted(recv) == list(range(self.cells_local))

    def _cells(self, buf: torch.Tensor, C_alloc: int) -> torch.Tensor:
        return buf.reshape(self.cells_local, C_alloc * buf.shape[-1])

    def dispatch(self, send_local: torch.Tensor, C_alloc: int, group=None) -> torch.Tensor:
        """Local slice of the SEND-layout buffer -> local slice of the RECV-layout buffer (rows of my experts)."""
        cells = self._cells(send_local, C_alloc)
        out_of_order = cells.index_select(0, self.send_cells.to(cells.device)).contiguous()
        arrived = torch.empty_like(out_of_order)
        dist.all_to_all_single(arrived, out_of_order, group=group)
        recv = torch.empty_like(arrived)
        recv.index_copy_(0, self.recv_cells.to(cells.device), arrived)
        return recv.reshape(send_local.shape)

    def combine(self, recv_local: torch.Tensor, C_alloc: int, group=None) -> torch.Tensor:
        """The way back: expert outputs in RECV layout -> SEND layout on the ranks the tokens came from."""
        cells = self._cells(recv_local, C_alloc)
        leaving = cells.index_select(0, self.recv_cells.to(cells.device)).contiguous()
        arrived = torch.empty_like(leaving)
        dist.all_to_all_single(arrived, leaving, group=group)
        send = torch.empty_like(arrived)
        send.index_copy_(0, self.send_cells.to(cells.device), arrived)
        return send.reshape(recv_local.shape)


class PeerBuffers:
    """Receive buffers of all ranks, addressable from every rank, for the fused dispatch / combine calls.

    Rank q holds the rows [q * R, (q + 1) * R) of the global receive-side buffer (R = rows_per_rank).  With one rank
    the buffer is an ordinary tensor.  With several, it is allocated as torch symmetric memory, whose rendezvous
    hands every rank a pointer to every peer's buffer (a peer mapping over NVLink); ``pointers`` is the table the
    C-ABI calls take.  ``barrier()`` orders the steps across ranks: call it (after synchronising the stream that ran
    the kernels) between dispatch, the experts and combine.  No multicast mapping is created or used.
    """

    def __init__(self, rows_per_rank: int, H: int, dtype: torch.dtype, device, group=None):
        self.group = group
        world = dist.get_world_size(group) if dist.is_available() and dist.is_initialized() else 1
        self.world = world
        if world == 1:
            self.local = torch.empty(rows_per_rank, H, dtype=dtype, device=device)
            self.pointers = [self.local.data_ptr()]
            self._handle = None
        else:
            import torch.distributed._symmetric_memory as symm
            self.local = symm.empty(rows_per_rank, H, dtype=dtype, device=device)
            self._handle = symm.rendezvous(self.local, group=group if group is not None else dist.group.WORLD)
            self.pointers = [int(p) for p in self._handle.buffer_ptrs]

    @classmethod
    def from_mappings(cls, local: torch.Tensor, pointers, group=None):
        """Buffers whose peer mappings the caller obtained some other way (CUDA IPC handles, a driver-level
        mapping): ``local`` is this rank's slice, ``pointers[q]`` the address of rank q's slice as valid on THIS GPU
        (``pointers[rank]`` = ``local.data_ptr()``).  Same barrier / ordering behaviour as the symmetric-memory form."""
        self = cls.__new__(cls)
        self.group = group
        self.world = len(pointers)
        self.local = local
        self.pointers = [int(p) for p in pointers]
        self._handle = None
        return self

    def synchronize(self, stream=None):
        """Waits for the stream that ran this rank's kernels (before the host reads their results or meets its peers)."""
        (stream or torch.cuda.current_stream()).synchronize()

    def barrier(self, stream=None):
        if self.world == 1:
            return
        self.synchronize(stream)
        dist.barrier(group=self.group)

    def order(self, first, then):
        """Work queued on stream ``then`` from now on starts after everything queued on ``first`` so far."""
        (then or torch.cuda.current_stream()).wait_stream(first or torch.cuda.current_stream())


def peer_layer_forward(B, sharding, shape_local, C_alloc, rule, x, src_dev, recv: "PeerBuffers", y: "PeerBuffers",
                       st, w_in=None, w_out=None, F=0, h1=None, out=None, group=None, stream=None, mark=None,
                       slices=1, ffn_stream=None):
    """One MoE layer pass on this rank with the exchange fused into dispatch and combine.

    ``shape_local`` describes the WHOLE logical map with ``T`` = this rank's tokens and the receive-side layout;
    ``x`` / ``src_dev`` are this rank's tokens and their (global) source devices; ``st`` is a ``binding.RouterState``
    for ``shape_local``; ``recv`` / ``y`` hold every rank's slice of the receive-side buffer and of the expert
    outputs (``y`` may be ``recv`` itself for identity experts).  ``w_in`` / ``w_out`` are the weights of THIS
    rank's experts ([E / world][F][H] and [E / world][H][F]).  Sequence: gate -> per-rank minima -> batch-wide
    capacity (All-Reduce MIN / SUM on the host side of ``sharding.global_capacity_inputs``) -> route -> peer-store
    dispatch -> barrier -> local experts -> barrier -> peer-load combine.  Only call sequencing lives here.

    Ordering across ranks (no kernel waits on another GPU, so the host orders the steps): the first barrier ends
    every rank's stores into the receive buffers before any expert reads them; the second ends every expert's
    writes of ``y`` before any combine loads them.  A rank's next pass begins with kernels that touch only its own
    memory and reaches its first barrier only after its own combine has completed, so with a separate ``y`` no
    third barrier is needed: the experts of the next pass cannot overwrite ``y`` before every rank's combine is
    done.  When ``y`` IS ``recv`` (identity experts), the next pass's peer stores would land in rows a slower rank's
    combine is still loading; a trailing barrier closes that window.  ``mark`` (optional) is called between the
    stages -- before and after the gate, after the route, after the dispatch and its barrier, after the experts and
    their barrier, after the combine -- so that a benchmark can record events there.

    ``slices`` > 1 (with experts) overlaps the exchange with the expert computation, as Sec. 3.2.4 describes: this
    rank's experts are cut into ``slices`` equal blocks; block s of EVERY rank's receive buffer is filled (windowed
    peer stores on ``stream``, then the barrier), and the experts of block s start on ``ffn_stream`` while block
    s + 1 is being stored.  The results are those of the unsliced pass, bit for bit.
    """
    mark = mark or (lambda: None)
    world = recv.world
    rank = dist.get_rank(group) if world > 1 else 0
    D = shape_local.D
    devs = sharding.devices_of_rank(D, world, rank)
    out = st.out if out is None else out
    mark()
    B.locmoe_gate(shape_local, x, None, st.idx, st.gate_w, st.cos_sim, None, stream)
    mark()
    rule_g = rule
    if world > 1:
        # the whole batch's rule: per-rank minima, then All-Reduce MIN / SUM across the ranks (host side)
        B.locmoe_capacity(shape_local, st.idx, st.cos_sim, rule, st.delta_e, st.theta_e, st.cap_dev, st.ws, stream)
        recv.synchronize(stream)      # the per-expert minima are read by the host-side reduction
        delta, T_global = sharding.global_capacity_inputs(st.delta_e, shape_local.T, group)
        rule_g = B.CapacityRule(rule.min_mult, rule.capacity_factor, delta if rule.delta_override < 0 else rule.delta_override,
                                rule.bound_form, T_global)
    # (one rank: its tokens are the batch, the fused call measures delta itself and nothing is read back)
    B.locmoe_capacity_route(shape_local, st.idx, st.cos_sim, src_dev, rule_g, st.delta_e, st.theta_e, st.cap_dev, C_alloc,
                            st.pos, st.slot, st.drop, st.inv, st.counts, st.kept, st.send_counts, st.load, st.locality,
                            st.status, st.ws, stream)
    mark()
    ydt = B.dtype_code(y.local.dtype)
    E_loc = shape_local.E // world
    if w_in is not None and slices > 1:
        if E_loc % slices:
            raise ValueError("a rank's %d experts do not split into %d equal blocks" % (E_loc, slices))
        Eb = E_loc // slices                      # experts per block
        Rb = Eb * D * C_alloc                     # rows of a block inside a rank's buffer
        sh_ffn = B.make_shape(shape_local.T, shape_local.H, Eb, 1, 1, recv.local.dtype, B.LAYOUT_RECV)
        for s in range(slices):
            B.locmoe_dispatch_peer(shape_local, C_alloc, x, st.inv, st.slot, recv.pointers, devs.start, devs.stop, True,
                                   stream, window=(s * Rb, (s + 1) * Rb))
            recv.barrier(stream)                  # block s of every rank's buffer is complete
            recv.order(stream, ffn_stream)        # (one rank: no barrier, the streams alone order the two steps)
            B.locmoe_expert_ffn(sh_ffn, D * C_alloc, F, recv.local[s * Rb:(s + 1) * Rb], w_in[s * Eb:(s + 1) * Eb],
                                w_out[s * Eb:(s + 1) * Eb], h1[s * Rb:(s + 1) * Rb], y.local[s * Rb:(s + 1) * Rb], ffn_stream)
        mark()
        y.barrier(ffn_stream)
        y.order(ffn_stream, stream)
    else:
        B.locmoe_dispatch_peer(shape_local, C_alloc, x, st.inv, st.slot, recv.pointers, devs.start, devs.stop, True, stream)
        recv.barrier(stream)
        mark()
        if w_in is not None:
            # this rank's experts on its slice of the receive buffer: a shape whose experts are the local ones
            # (one logical device holding E / world experts with D * C_alloc rows each: the same rows, regrouped)
            sh_ffn = B.make_shape(shape_local.T, shape_local.H, E_loc, 1, 1, recv.local.dtype, B.LAYOUT_RECV)
            B.locmoe_expert_ffn(sh_ffn, D * C_alloc, F, recv.local, w_in, w_out, h1, y.local, stream)
        y.barrier(stream)
    mark()
    B.locmoe_combine_peer(shape_local, C_alloc, y.pointers, ydt, st.slot, st.gate_w, out, stream)
    mark()
    if world > 1 and (y is recv or y.local.data_ptr() == recv.local.data_ptr()):
        y.barrier(stream)   # the next pass's peer stores must not overtake a slower rank's loads of the same rows
    return out
