"""Two CPU ranks over gloo: one equal-split All-to-All turns the send-side buffers of all ranks into the
receive-side (per-expert) buffers, and back.  Expected buffers come from the oracle's two layouts."""
import os
import socket
import sys

import numpy as np
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


def _worker(rank, world, port, N, Dn, E, q):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import oracle
    from paper_2401_13920_b200.exchange import ExchangePlan
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        T, H, C = 1500, 12, 9
        D = N * Dn
        rng = np.random.default_rng(5)                      # the same global batch on every rank
        x = rng.standard_normal((T, H)).astype(np.float32)
        idx = rng.integers(0, E, T).astype(np.int32)
        src = rng.integers(0, D, T).astype(np.int32)
        rows = D * E * C
        send = oracle.dispatch(x, 0, oracle.route(idx, src, E, N, Dn, C, C, 0).slot, rows)
        recv = oracle.dispatch(x, 0, oracle.route(idx, src, E, N, Dn, C, C, 1).slot, rows)
        per = rows // world
        mine_send = torch.from_numpy(send[rank * per:(rank + 1) * per].copy())   # rows of my source devices
        mine_recv = torch.from_numpy(recv[rank * per:(rank + 1) * per].copy())   # rows of my experts
        plan = ExchangePlan(N, Dn, E, world, rank)
        got = plan.dispatch(mine_send, C)
        ok = bool(torch.equal(got, mine_recv))
        back = plan.combine(got, C)
        ok &= bool(torch.equal(back, mine_send))
        q.put((rank, ok))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("N,Dn,E", [(2, 2, 4), (2, 4, 16), (1, 2, 6)])
def test_all_to_all_turns_send_layout_into_recv_layout(oracle_mod, N, Dn, E):
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, N, Dn, E, q)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(timeout=120)
    res = sorted(q.get(timeout=5) for _ in range(2))
    assert res == [(0, True), (1, True)]


def test_single_rank_plan_is_the_layout_permutation(oracle_mod):
    # world = 1: no communication needed, the two index lists alone map SEND cells to RECV cells
    sys.path.insert(0, ROOT)
    from paper_2401_13920_b200.exchange import ExchangePlan
    N, Dn, E, C, H, T = 2, 2, 8, 5, 6, 400
    D = N * Dn
    rng = np.random.default_rng(6)
    x = rng.standard_normal((T, H)).astype(np.float32)
    idx = rng.integers(0, E, T).astype(np.int32)
    src = rng.integers(0, D, T).astype(np.int32)
    rows = D * E * C
    send = oracle_mod.dispatch(x, 0, oracle_mod.route(idx, src, E, N, Dn, C, C, 0).slot, rows)
    recv = oracle_mod.dispatch(x, 0, oracle_mod.route(idx, src, E, N, Dn, C, C, 1).slot, rows)
    plan = ExchangePlan(N, Dn, E, 1, 0)
    cells = torch.from_numpy(send).reshape(plan.cells_local, C * H)
    out = torch.empty_like(cells)
    out.index_copy_(0, plan.recv_cells, cells.index_select(0, plan.send_cells))
    assert np.array_equal(out.reshape(rows, H).numpy(), recv)
