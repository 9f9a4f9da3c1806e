"""Two CPU ranks over gloo: the path shards by source device with no exchange step.

Each rank routes (with the oracle) only the tokens of its own logical source
devices; positions, drops and slots must equal those of the whole batch and
the count matrices of the ranks must add up to the global ones.  Also covers
the bench's max-over-ranks timing helper."""
import os
import socket
import sys

import numpy as np
import pytest
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, layout, q):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import oracle
    from paper_2401_13920_b200 import sharding
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        T, E, N, Dn, C = 3000, 16, 2, 4, 20
        D = N * Dn
        rng = np.random.default_rng(77)            # same stream on both ranks: the same global batch
        idx = rng.integers(0, E, T).astype(np.int32)
        src = rng.integers(0, D, T).astype(np.int32)
        whole = oracle.route(idx, src, E, N, Dn, C, C, layout)
        mine = sharding.shard_by_source(src, D, world, rank)
        part = oracle.route(idx[mine], src[mine], E, N, Dn, C, C, layout)
        ok = True
        ok &= bool(np.array_equal(part.pos, whole.pos[mine]))
        ok &= bool(np.array_equal(part.drop, whole.drop[mine]))
        ok &= bool(np.array_equal(part.slot, whole.slot[mine]))          # same row in the global buffer
        counts = sharding.sum_over_ranks(part.counts)
        sends = sharding.sum_over_ranks(part.send_counts)
        loc = sharding.sum_over_ranks(part.locality)
        load = sharding.sum_over_ranks(part.load)
        ok &= bool(np.array_equal(counts, whole.counts)) and bool(np.array_equal(sends, whole.send_counts))
        ok &= bool(np.array_equal(loc, whole.locality)) and bool(np.array_equal(load, whole.load))
        # a rank only fills rows of its own source devices (SEND layout) -- disjoint row sets
        occupied = sharding.sum_over_ranks((part.inv >= 0).astype(np.int64))
        ok &= bool(occupied.max() <= 1) and int(occupied.sum()) == int((whole.inv >= 0).sum())
        # capacity of the whole batch from per-rank minima: every rank gets the batch-wide delta and token count
        import torch
        de = torch.full((E,), 1.0)
        de[rank] = 0.25 - 0.5 * rank                  # rank 1 holds a negative minimum: clamped to 0
        de[5] = 0.125 + rank
        delta, Tg = sharding.global_capacity_inputs(de, len(mine))
        ok &= delta == 0.0 and Tg == T
        delta2, _ = sharding.global_capacity_inputs(torch.full((E,), 0.5 + 0.25 * rank), 1)
        ok &= delta2 == 0.5
        # timing helper: the slowest rank decides
        slow = sharding.max_over_ranks(10.0 + 5.0 * rank)
        thr = sharding.aggregate_throughput(1000, 4, 10.0 + 5.0 * rank, world)
        ok &= slow == 15.0 and abs(thr - world * 1000 * 4 / 15e-3) < 1e-6
        q.put((rank, ok))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("layout", [0, 1])
def test_two_ranks_shard_by_source_device(layout, oracle_mod):
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, layout, q)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(timeout=120)
    res = sorted(q.get(timeout=5) for _ in range(2))
    assert res == [(0, True), (1, True)]
    assert all(p.exitcode == 0 for p in procs)


def test_device_blocks():
    sys.path.insert(0, ROOT)
    from paper_2401_13920_b200 import sharding
    assert list(sharding.devices_of_rank(8, 2, 1)) == [4, 5, 6, 7]
    with pytest.raises(ValueError):
        sharding.devices_of_rank(6, 4, 0)
    src = np.array([0, 5, 3, 7, 4, 1])
    assert sharding.shard_by_source(src, 8, 2, 0).tolist() == [0, 2, 5]
    assert sharding.shard_by_source(src, 8, 2, 1).tolist() == [1, 3, 4]
