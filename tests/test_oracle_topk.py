"""Pins of the oracle's top-k variant (gate and combine)."""
import numpy as np
import pytest

import oracle


def _tokens(T, H, seed):
    return np.random.default_rng(seed).standard_normal((T, H)).astype(np.float32)


def test_k1_is_the_top1_gate():
    x = _tokens(500, 64, 1)
    g = oracle.gate(x, oracle.F32, 8)
    idx_k, R_k, gap = oracle.gate_topk(x, oracle.F32, 8, 1)
    assert np.array_equal(idx_k[0], g.idx) and np.array_equal(R_k[0], g.R)
    assert np.allclose(gap, g.gap, rtol=0, atol=0)


@pytest.mark.parametrize("K", [2, 3, 8])
def test_choices_are_the_k_largest_logits_in_order(K):
    E = 8
    x = _tokens(800, 96, 2)
    eps = np.linspace(-0.1, 0.1, E).astype(np.float32)
    g = oracle.gate(x, oracle.F32, E, eps=eps, want_G=True, want_probs=True)
    idx_k, R_k, gap = oracle.gate_topk(x, oracle.F32, E, K, eps=eps)
    order = np.argsort(-g.G, axis=1, kind="stable")[:, :K]          # descending, ties to the lower index
    assert np.array_equal(idx_k.T, order)
    assert np.allclose(R_k.T, np.take_along_axis(g.probs, order, 1), rtol=1e-15)
    assert (np.diff(R_k, axis=0) <= 0).all() and (R_k.sum(0) <= 1 + 1e-12).all()
    if K == E:
        assert np.allclose(R_k.sum(0), 1.0, rtol=1e-13)
    srt = -np.sort(-g.G, axis=1)
    want_gap = np.min(srt[:, :min(K, E - 1)] - srt[:, 1:min(K, E - 1) + 1], axis=1)
    assert np.allclose(gap, want_gap, rtol=0, atol=1e-15)


def test_ties_go_to_the_lower_index_hand_example():
    # groups of 2: means (1, 3, 3, 0) -> choices 1, 2 (tie between 1 and 2, lower first), then 0
    x = np.array([[1, 1, 3, 3, 3, 3, -5, 5]], np.float32)
    idx_k, R_k, gap = oracle.gate_topk(x, oracle.F32, 4, 3)
    assert list(idx_k[:, 0]) == [1, 2, 0]
    den = 2 * np.exp(3) + np.exp(1) + 1
    assert np.allclose(R_k[:, 0], [np.exp(3) / den, np.exp(3) / den, np.exp(1) / den], rtol=1e-15)
    assert gap[0] == 0.0


def test_combine_topk_is_the_sum_of_top1_combines_and_handles_drops():
    rng = np.random.default_rng(4)
    T, H, rows, K = 50, 12, 40, 2
    y = rng.standard_normal((rows, H)).astype(np.float32)
    slot = rng.integers(0, rows, size=(K, T)).astype(np.int32)
    slot[0, ::5] = -1
    slot[1, ::7] = -1                         # token 0 and token 35 lose both choices
    R = rng.random((K, T))
    got = oracle.combine_topk(y, oracle.F32, slot, R)
    want = sum(oracle.combine(y, oracle.F32, slot[c], R[c]) for c in range(K))
    assert np.allclose(got, want, rtol=1e-15, atol=0)
    both_dropped = (slot < 0).all(0)
    assert both_dropped.any() and not got[both_dropped].any()
    # brute force on one element
    t = int(np.nonzero((slot >= 0).all(0))[0][0])
    assert np.isclose(got[t, 5], R[0, t] * float(y[slot[0, t], 5]) + R[1, t] * float(y[slot[1, t], 5]), rtol=1e-15)


def test_constant_expert_rows_give_the_sum_of_scores():
    x = _tokens(64, 32, 7)
    idx_k, R_k, _ = oracle.gate_topk(x, oracle.F32, 4, 2)
    y = np.full((10, 6), 2.0, np.float32)
    slot = np.zeros((2, 64), np.int32)
    out = oracle.combine_topk(y, oracle.F32, slot, R_k)
    assert np.allclose(out, 2.0 * R_k.sum(0)[:, None], rtol=1e-15)
