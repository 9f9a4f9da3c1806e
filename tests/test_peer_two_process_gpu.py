"""The fused exchange with TWO real ranks: two processes (a gloo group) that share the one GPU of the test box, each
owning half of the logical devices and half of the receive buffer; a rank sees the other's half through a CUDA IPC
mapping (torch hands CUDA tensors between processes that way), so its peer stores and peer loads really go through a
pointer that belongs to another process.  No kernel waits on another (the host orders the steps with barriers), so
sharing a GPU is safe.  `exchange.peer_layer_forward` runs with world = 2 -- host All-Reduce of the minima, batch-wide
capacity, barriers, and (one case) the exchange overlapped with the experts block by block -- and every rank's slice of the receive buffer, its routing and its combined output must equal, bit
for bit, those of the whole batch routed by one process."""
import os
import socket
import sys

import pytest
import torch
import torch.multiprocessing as mp

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, to_peer, from_peer, results, with_ffn, slices):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from paper_2401_13920_b200 import binding as B, exchange, sharding, workloads as W
        dev = torch.device("cuda:0")
        torch.cuda.set_device(0)
        w = W.CONFIGS[5].scaled(6000)
        F = 512
        x_all, src_all = W.make_tokens(w, dev), W.make_src(w, dev)           # the same seeded batch in both processes
        D = w.n_nodes * w.dev_per_node
        sel = torch.as_tensor(sharding.shard_by_source(src_all.cpu().numpy(), D, world, rank), device=dev)
        x, src = x_all[sel].contiguous(), src_all[sel].contiguous()
        sh = B.make_shape(len(sel), w.H, w.E, w.n_nodes, w.dev_per_node, x.dtype, B.LAYOUT_RECV)
        rule = B.CapacityRule(1.0, 1.0, -1.0, 0, 0)
        Ca = B.conventional_capacity(w.T, D, w.E, 1.0)
        rows = D * w.E * Ca
        rpr = rows // world
        # my halves of the receive buffer and of the expert outputs; the peer's halves arrive as IPC mappings
        mine = [torch.full((rpr, w.H), 3.0, dtype=x.dtype, device=dev), torch.full((rpr, w.H), 5.0, dtype=torch.bfloat16, device=dev)]
        to_peer.put(mine)
        theirs = from_peer.get(timeout=120)
        def table(i):
            t = [None, None]
            t[rank], t[1 - rank] = mine[i].data_ptr(), theirs[i].data_ptr()
            return t
        recv = exchange.PeerBuffers.from_mappings(mine[0], table(0))
        yb = exchange.PeerBuffers.from_mappings(mine[1], table(1)) if with_ffn else recv
        w_in = w_out = h1 = None
        if with_ffn:
            w_all_in, w_all_out = W.make_expert_weights(w, F, dev)
            El = w.E // world
            w_in, w_out = w_all_in[rank * El:(rank + 1) * El].contiguous(), w_all_out[rank * El:(rank + 1) * El].contiguous()
            h1 = torch.empty(rpr, F, dtype=torch.bfloat16, device=dev)
        st = B.make_router(sh, Ca, rule, dev, with_buffer=False)
        out = torch.empty(len(sel), w.H, dtype=x.dtype, device=dev)
        exchange.peer_layer_forward(B, sharding, sh, Ca, rule, x, src, recv, yb, st, w_in, w_out, F, h1, out=out, slices=slices,
                                    ffn_stream=torch.cuda.Stream(dev) if slices > 1 else None)
        torch.cuda.synchronize()
        dist.barrier()
        # the whole batch in one process: the reference every rank compares its share with
        shg = B.make_shape(w.T, w.H, w.E, w.n_nodes, w.dev_per_node, x.dtype, B.LAYOUT_RECV)
        stg = B.make_router(shg, Ca, rule, dev)
        want = torch.empty(w.T, w.H, dtype=x.dtype, device=dev)
        if with_ffn:
            h1g = torch.empty(rows, F, dtype=torch.bfloat16, device=dev)
            yg = torch.empty(rows, w.H, dtype=torch.bfloat16, device=dev)
            B.locmoe_moe_layer(shg, x_all, src_all, None, rule, Ca, F, w_all_in, w_all_out, B.layer_buffers(stg, h1g, yg), want)
        else:
            B.locmoe_moe_layer(shg, x_all, src_all, None, rule, Ca, 0, None, None, B.layer_buffers(stg), want)
        torch.cuda.synchronize()
        capg, cap = B.locmoe_capacity_read(stg.cap_dev), B.locmoe_capacity_read(st.cap_dev)
        checks = {
            "capacity": (cap.C_local, cap.C_expert, cap.delta) == (capg.C_local, capg.C_expert, capg.delta),
            "slot": bool(torch.equal(st.slot, stg.slot[sel])),
            "buffer": bool(torch.equal(mine[0].view(torch.int16), stg.buf[rank * rpr:(rank + 1) * rpr].view(torch.int16))),
            "out": bool(torch.equal(out.view(torch.int16), want[sel].view(torch.int16))),
            "flags": B.locmoe_device_flags() == 0,
            "drops_and_keeps": 0 < int((st.slot < 0).sum()) < len(sel),
        }
        results.put((rank, checks))
        dist.barrier()          # the peer may still be reading my buffers through its mapping
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("with_ffn,slices", [(False, 1), (True, 1), (True, 4)])
def test_two_ranks_sharing_one_gpu_exchange_through_ipc_mappings(with_ffn, slices):
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    q01, q10, results = ctx.Queue(), ctx.Queue(), ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(0, 2, port, q01, q10, results, with_ffn, slices)),
             ctx.Process(target=_worker, args=(1, 2, port, q10, q01, results, with_ffn, slices))]
    for p in procs:
        p.start()
    got = sorted(results.get(timeout=300) for _ in range(2))
    for p in procs:
        p.join(timeout=120)
    assert [p.exitcode for p in procs] == [0, 0]
    for rank, checks in got:
        assert all(checks.values()), (rank, checks)
