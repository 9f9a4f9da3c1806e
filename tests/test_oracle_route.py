"""Pins for the oracle's route, dispatch and combine stages: capacity-bounded
first-come-first-served placement (Sec. 3.2.3), All-to-All shaped buffer with
intra-node destinations first (abstract, Sec. 3.2.4), and y_m = R_m * expert
output (first equation of Sec. 3.2.1)."""
import numpy as np
import pytest

F32, BF16 = 0, 1
SEND, RECV = 0, 1


def _rank_py(a, b, N, Dn):
    return ((b // Dn - a // Dn) % N) * Dn + ((b % Dn - a % Dn) % Dn)


def test_destination_order_is_intra_node_first(oracle_mod):
    for N, Dn in [(2, 2), (2, 4), (8, 8), (1, 4), (3, 1)]:
        D = N * Dn
        r = oracle_mod.dest_order(N, Dn)
        for a in range(D):
            assert sorted(r[a]) == list(range(D))          # a permutation of the destinations
            assert r[a, a] == 0                            # self first
            for b in range(D):
                assert (r[a, b] < Dn) == (a // Dn == b // Dn)   # own node before any other node
    # 2 nodes x 2 devices, destination lists ordered by rank
    r = oracle_mod.dest_order(2, 2)
    order = [list(np.argsort(r[a])) for a in range(4)]
    assert order == [[0, 1, 2, 3], [1, 0, 3, 2], [2, 3, 0, 1], [3, 2, 1, 0]]


def test_tiny_case_worked_by_hand(oracle_mod):
    # N = 2 nodes x 2 devices, 4 experts (one per device), one slot per (source, expert).
    idx = [2, 2, 0, 3, 2, 0, 1, 2]
    src = [0, 1, 0, 3, 0, 2, 1, 1]
    # tokens 4 and 7 repeat the (src, expert) pairs of tokens 0 and 1 -> second in queue -> dropped.
    s = oracle_mod.route(idx, src, 4, 2, 2, 1, 1, SEND)
    assert list(s.pos) == [0, 0, 0, 0, 1, 0, 0, 1]
    assert list(s.drop) == [0, 0, 0, 0, 1, 0, 0, 1]
    # SEND row = (src * 4 + rank(src -> dev)) * 1 + pos
    assert list(s.slot) == [2, 7, 0, 12, -1, 10, 4, -1]
    r = oracle_mod.route(idx, src, 4, 2, 2, 1, 1, RECV)
    # RECV row = (expert * 4 + rank(dev -> src)) * 1 + pos
    assert list(r.slot) == [10, 11, 0, 12, -1, 2, 4, -1]
    assert s.send_counts.tolist() == [[1, 0, 1, 0], [0, 1, 1, 0], [1, 0, 0, 0], [0, 0, 0, 1]]
    assert s.locality.tolist() == [[3, 0, 5], [3, 0, 3]]
    assert s.load.tolist() == [2, 1, 4, 1]
    assert s.counts[0].tolist() == [1, 0, 2, 0] and s.kept[0].tolist() == [1, 0, 1, 0]


@pytest.mark.parametrize("layout", [SEND, RECV])
@pytest.mark.parametrize("T,E,N,Dn,C", [(300, 8, 2, 2, 3), (512, 12, 3, 2, 40), (257, 4, 1, 4, 1), (64, 16, 2, 4, 2)])
def test_route_against_brute_force_definition(oracle_mod, layout, T, E, N, Dn, C):
    rng = np.random.default_rng(20 + T)
    D = N * Dn
    Ed = E // D
    idx = rng.integers(0, E, T).astype(np.int32)
    src = rng.integers(0, D, T).astype(np.int32)
    out = oracle_mod.route(idx, src, E, N, Dn, C, C + 2, layout)
    # pos from its definition, written here independently (and by the oracle's own O(T^2) loop)
    pos = np.array([sum(1 for u in range(t) if src[u] == src[t] and idx[u] == idx[t]) for t in range(T)])
    assert np.array_equal(out.pos, pos)
    assert np.array_equal(oracle_mod.pos_bruteforce(idx, src), pos)
    assert np.array_equal(out.drop, pos >= C)
    Ca = C + 2
    for t in range(T):
        if pos[t] >= C:
            assert out.slot[t] == -1
            continue
        b, el, s = idx[t] // Ed, idx[t] % Ed, src[t]
        if layout == SEND:
            row = ((s * D + _rank_py(s, b, N, Dn)) * Ed + el) * Ca + pos[t]
        else:
            row = ((b * Ed + el) * D + _rank_py(b, s, N, Dn)) * Ca + pos[t]
        assert out.slot[t] == row
    # structure
    keep = out.slot >= 0
    assert len(set(out.slot[keep])) == keep.sum()                    # all slots distinct
    assert np.array_equal(out.inv[out.slot[keep]], np.nonzero(keep)[0])   # inv o slot = id
    assert (out.inv >= 0).sum() == keep.sum()
    cnt = np.zeros((D, E), np.int64)
    np.add.at(cnt, (src, idx), 1)
    assert np.array_equal(out.counts, cnt)
    assert np.array_equal(out.kept, np.minimum(cnt, C))
    assert out.kept.max() <= C                                      # nobody exceeds the capacity
    assert out.kept.sum() + out.drop.sum() == T
    assert np.array_equal(out.load, cnt.sum(0))
    assert (out.kept.sum(0) <= D * C).all()
    assert np.array_equal(out.send_counts, out.kept.reshape(D, D, Ed).sum(2))
    assert out.locality[0].sum() == T and out.locality[1].sum() == keep.sum()
    dev = idx // Ed
    assert out.locality[0, 0] == (dev == src).sum()
    assert out.locality[0, 1] == ((dev // Dn == src // Dn) & (dev != src)).sum()
    assert out.locality[1, 2] == ((dev // Dn != src // Dn) & keep).sum()
    assert out.status == 0


def test_single_source_slot_order_is_a_stable_sort(oracle_mod):
    # One source device and ample capacity: reading the SEND buffer front to back lists the tokens
    # sorted stably by (destination rank, local expert) -- the library's stable argsort.
    rng = np.random.default_rng(30)
    T, E, N, Dn = 400, 8, 2, 2
    D, Ed = 4, 2
    idx = rng.integers(0, E, T).astype(np.int32)
    src = np.full(T, 3, np.int32)
    out = oracle_mod.route(idx, src, E, N, Dn, T, T, SEND)
    key = np.array([_rank_py(3, e // Ed, N, Dn) * Ed + e % Ed for e in idx])
    order = np.argsort(key, kind="stable")
    assert np.array_equal(out.inv[out.inv >= 0], order)
    assert out.drop.sum() == 0


def test_clamp_and_bad_source(oracle_mod):
    idx = np.array([0, 0, 0, 1, 1], np.int32)
    src = np.array([0, 0, 0, 9, -1], np.int32)
    out = oracle_mod.route(idx, src, 2, 1, 2, 5, 2, SEND)       # C_local 5 > C_alloc 2 -> clamped to 2
    assert out.status == 1 | 2
    assert list(out.drop) == [0, 0, 1, 1, 1]
    assert list(out.pos) == [0, 1, 2, -1, -1]
    assert out.counts.sum() == 3 and out.load.tolist() == [3, 0]


def test_dispatch_combine_round_trip(oracle_mod):
    # Identity experts and unit scores: combine(dispatch(x)) returns x for every kept token, 0 otherwise.
    rng = np.random.default_rng(40)
    T, H, E, N, Dn, C = 600, 48, 8, 2, 4, 8
    x = rng.standard_normal((T, H)).astype(np.float32)
    idx = rng.integers(0, E, T).astype(np.int32)
    src = rng.integers(0, N * Dn, T).astype(np.int32)
    for layout in (SEND, RECV):
        rt = oracle_mod.route(idx, src, E, N, Dn, C, C, layout)
        rows = N * Dn * E * C
        buf = oracle_mod.dispatch(x, F32, rt.slot, rows)
        keep = rt.slot >= 0
        assert 0 < keep.sum() < T
        assert np.array_equal(buf[rt.slot[keep]], x[keep])
        empty = np.ones(rows, bool)
        empty[rt.slot[keep]] = False
        assert not buf[empty].any()
        assert np.allclose(buf.astype(np.float64).sum(0), x[keep].astype(np.float64).sum(0), atol=1e-9)
        back = oracle_mod.combine(buf, F32, rt.slot, np.ones(T))
        assert np.array_equal(back[keep], x[keep].astype(np.float64))
        assert not back[~keep].any()


def test_combine_scales_by_the_score(oracle_mod):
    # y_m = R_m * (expert output of the chosen expert); bf16 expert outputs are widened exactly.
    y32 = np.array([[1.0, -2.0, 0.5, 4.0], [8.0, 0.25, -1.0, 3.0], [7.0, 7.0, 7.0, 7.0]], np.float32)
    ybits = (y32.view(np.uint32) >> 16).astype(np.uint16)        # exactly representable values
    slot = np.array([1, -1, 0, 2], np.int32)
    R = np.array([0.5, 0.9, 0.125, 1.0])
    out = oracle_mod.combine(ybits, BF16, slot, R)
    assert np.array_equal(out, [[4.0, 0.125, -0.5, 1.5], [0, 0, 0, 0], [0.125, -0.25, 0.0625, 0.5], [7, 7, 7, 7]])
    prev = np.ones((4, 4))
    out2 = oracle_mod.combine(y32, F32, slot, R, prev=prev)
    assert np.array_equal(out2, out + 1.0)
