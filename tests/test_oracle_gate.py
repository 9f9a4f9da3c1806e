"""Pins for the oracle's gate (Sec. 3.2.1: GrAP weight, ReLU, softmax, arg-max,
score; Lemma 1, Lemma 2).  Each test states the fact it pins; none of them
re-types the oracle's own loop."""
import numpy as np
import pytest
from scipy.special import softmax
from scipy.stats import chi2

F32, BF16 = 0, 1


def _bf16_round(x32: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bits (round to nearest even), library-free bit trick."""
    u = np.ascontiguousarray(x32, dtype=np.float32).view(np.uint32)
    r = ((u >> 16) & 1) + 0x7FFF
    return ((u + r) >> 16).astype(np.uint16)


def test_grap_weight_is_block_average_and_orthogonal(oracle_mod):
    # Sec. 3.2.1: w_i = (n/d) 1{i d/n <= j < (i+1) d/n}; the paper notes that these weights are mutually orthogonal;
    # Assumption 1: equal norms.
    for n, d in [(8, 1024), (64, 5120), (256, 5120), (4, 12), (1, 7)]:
        W = oracle_mod.grap_weight(n, d)
        g = d // n
        expect = np.kron(np.eye(n), np.ones((1, g))) * (n / d)
        assert np.array_equal(W, expect)
        gram = W @ W.T
        assert np.allclose(gram, np.eye(n) * (n / d), rtol=0, atol=1e-15)
        assert np.allclose(np.linalg.norm(W, axis=1), np.sqrt(n / d))


@pytest.mark.parametrize("T,H,E", [(64, 1024, 8), (33, 5120, 64), (17, 5120, 256), (9, 60, 5)])
def test_group_mean_equals_dense_layer_with_fixed_weight(oracle_mod, T, H, E):
    # Sec. 3.2.1 presents GrAP as a dense layer whose weight is fixed to w_i: G = ReLU(x W^T).
    rng = np.random.default_rng(1)
    x = rng.standard_normal((T, H)).astype(np.float32)
    W = np.kron(np.eye(E), np.ones((1, H // E))) * (E / H)
    out = oracle_mod.gate(x, F32, E, want_G=True, want_probs=True)
    dense = np.maximum(x.astype(np.float64) @ W.T, 0.0)
    assert np.allclose(out.G, dense, rtol=1e-13, atol=1e-15)
    # arg-max of softmax (Eq. max_expert) and the score (Eq. gating_score) via library softmax
    p = softmax(dense, axis=1)
    assert np.allclose(out.probs, p, rtol=1e-12, atol=0)
    assert np.allclose(out.probs.sum(1), 1.0, rtol=0, atol=1e-13)
    assert np.array_equal(out.idx, p.argmax(1))
    assert np.allclose(out.R, p[np.arange(T), out.idx], rtol=1e-12)
    srt = np.sort(dense, axis=1)
    assert np.allclose(out.gap, srt[:, -1] - srt[:, -2], rtol=0, atol=1e-15)


def test_bias_enters_before_relu(oracle_mod):
    # G = ReLU(w.x + eps): a large bias on expert 2 wins; a very negative bias is clamped to 0.
    x = np.zeros((2, 8), np.float32)
    x[0] = [1, 1, 0, 0, 0, 0, 0, 0]          # means: 1, 0, 0, 0
    x[1] = [0, 0, 0, 0, 0, 0, -4, -4]        # means: 0, 0, 0, -4
    eps = np.array([0.0, 0.0, 5.0, -3.0], np.float32)
    out = oracle_mod.gate(x, F32, 4, eps=eps, want_G=True)
    assert np.array_equal(out.G, [[1, 0, 5, 0], [0, 0, 5, 0]])
    assert np.array_equal(out.idx, [2, 2])
    # the cosine uses the raw weight and the raw token (no bias, no ReLU): token 0 is orthogonal to w_2
    assert out.cos[0] == 0.0


def test_hand_checkable_cases(oracle_mod):
    # E = 2, H = 4, groups {0,1} and {2,3}
    x = np.array([[1, 3, 2, 2],      # means 2, 2 -> tie -> lowest index, R = 1/2
                  [0, 0, 4, 0],      # means 0, 2 -> expert 1, R = 1/(1+e^-2), cos = 2/(sqrt(1/2)*4)
                  [-1, -1, -2, -2],  # all means <= 0 -> logits all 0 -> expert 0, R = 1/2, cos < 0
                  [0, 0, 0, 0]],     # zero token: cos defined as 0
                 np.float32)
    out = oracle_mod.gate(x, F32, 2)
    assert np.array_equal(out.idx, [0, 1, 0, 0])
    assert np.allclose(out.R, [0.5, 1 / (1 + np.exp(-2.0)), 0.5, 0.5], rtol=1e-15)
    assert np.allclose(out.cos, [2 / (np.sqrt(0.5) * np.sqrt(18)), 2 / (np.sqrt(0.5) * 4),
                                 -1 / (np.sqrt(0.5) * np.sqrt(10)), 0.0], rtol=1e-15)
    assert np.array_equal(out.gap, [0.0, 2.0, 0.0, 0.0])


def test_single_expert_and_all_zero_logits(oracle_mod):
    rng = np.random.default_rng(2)
    x = rng.standard_normal((5, 16)).astype(np.float32)
    out = oracle_mod.gate(x, F32, 1)
    assert np.array_equal(out.idx, np.zeros(5)) and np.array_equal(out.R, np.ones(5))
    out = oracle_mod.gate(-np.abs(x), F32, 8)
    assert np.array_equal(out.idx, np.zeros(5)) and np.allclose(out.R, 1 / 8)


def test_cosine_special_directions(oracle_mod):
    # Lemma 1 proof: <w_i, x> = |w_i||x| cos(theta).  x = c w_i -> cos = 1 and expert i;
    # x orthogonal to every w_i -> cos = 0.
    n, d = 8, 64
    g = d // n
    W = np.kron(np.eye(n), np.ones((1, g))) * (n / d)
    x = (3.5 * W).astype(np.float32)
    out = oracle_mod.gate(x, F32, n)
    assert np.array_equal(out.idx, np.arange(n))
    assert np.allclose(out.cos, 1.0, rtol=0, atol=1e-15)
    alt = np.tile(np.array([1.0, -1.0], np.float32), d // 2)[None, :]   # zero mean in every group
    out = oracle_mod.gate(alt, F32, n)
    assert out.cos[0] == 0.0
    rng = np.random.default_rng(3)
    out = oracle_mod.gate(rng.standard_normal((200, d)).astype(np.float32), F32, n)
    assert np.all(np.abs(out.cos) <= 1.0)


def test_lemma1_top1_is_minimum_angle(oracle_mod):
    # Lemma 1: with equal |w_i| the top-1 expert is the one at the smallest angle (largest cosine),
    # whenever at least one pre-activation is positive (ReLU otherwise flattens all logits to 0).
    rng = np.random.default_rng(4)
    T, H, E = 500, 640, 16
    x = rng.standard_normal((T, H)).astype(np.float32)
    W = np.kron(np.eye(E), np.ones((1, H // E))) * (E / H)
    xd = x.astype(np.float64)
    cosall = (xd @ W.T) / (np.linalg.norm(W, axis=1)[None, :] * np.linalg.norm(xd, axis=1)[:, None])
    out = oracle_mod.gate(x, F32, E)
    has_pos = cosall.max(1) > 0
    assert has_pos.sum() > 400
    assert np.array_equal(out.idx[has_pos], cosall.argmax(1)[has_pos])
    assert np.allclose(out.cos, cosall[np.arange(T), out.idx], rtol=1e-12, atol=1e-15)


def test_bf16_storage_is_widened_exactly(oracle_mod):
    rng = np.random.default_rng(5)
    x32 = rng.standard_normal((40, 320)).astype(np.float32)
    bits = _bf16_round(x32)
    widened = (bits.astype(np.uint32) << 16).view(np.float32)
    a = oracle_mod.gate(bits, BF16, 8, want_G=True)
    b = oracle_mod.gate(widened, F32, 8, want_G=True)
    assert np.array_equal(a.G, b.G) and np.array_equal(a.idx, b.idx)
    assert np.array_equal(a.R, b.R) and np.array_equal(a.cos, b.cos)


def test_lemma2_balanced_assignment_on_spherical_tokens(oracle_mod):
    # Lemma 2: P{i_j = i'} = 1/n for spherically symmetric tokens and orthogonal gates.
    rng = np.random.default_rng(6)
    T, H, E = 16384, 512, 16
    x = rng.standard_normal((T, H)).astype(np.float32)
    out = oracle_mod.gate(x, F32, E)
    load = np.bincount(out.idx, minlength=E)
    stat = ((load - T / E) ** 2 / (T / E)).sum()
    assert stat < chi2.ppf(0.9999, E - 1)


def test_shape_errors(oracle_mod):
    with pytest.raises(ValueError):
        oracle_mod.gate(np.zeros((2, 10), np.float32), F32, 3)


def test_aux_loss_definition_and_minimum(oracle_mod):
    # Sec. 3.2.2: L_aux = alpha n sum_i f_i P_i; under a uniform assignment with uniform probabilities the sum is
    # 1/n, so L_aux = alpha (the balanced case the paper names as the loss's minimum); alpha = 0.01.
    n, T = 8, 64
    idx = np.arange(T) % n
    probs = np.full((T, n), 1.0 / n)
    L, f, P = oracle_mod.aux_loss(idx, probs, 0.01)
    assert np.allclose(f, 1 / n) and np.allclose(P, 1 / n) and L == pytest.approx(0.01)
    # everything on one expert with probability one: f = P = e_0, L = alpha n
    probs = np.zeros((T, n)); probs[:, 0] = 1.0
    L, f, P = oracle_mod.aux_loss(np.zeros(T, np.int32), probs, 0.01)
    assert L == pytest.approx(0.01 * n)
    # against numpy on random data
    rng = np.random.default_rng(9)
    x = rng.standard_normal((500, 256)).astype(np.float32)
    g = oracle_mod.gate(x, F32, 16, want_probs=True)
    L, f, P = oracle_mod.aux_loss(g.idx, g.probs, 0.01)
    f_np = np.bincount(g.idx, minlength=16) / 500
    assert np.allclose(f, f_np) and np.allclose(P, g.probs.mean(0))
    assert L == pytest.approx(0.01 * 16 * (f_np * g.probs.mean(0)).sum(), rel=1e-12)


# ---- per-source-device bias table (the paper leaves eps_i undefined; a table indexed by the source device is one
#      reading of "locality-aware" bias, kept optional) ----

def test_per_source_bias_rows_by_hand(oracle_mod):
    # E = 2, H = 4: group means of [1, 1, 0.5, 0.5] are (1, 0.5).  Source 0 has no bias: expert 0 wins.
    # Source 1 lifts expert 1 by 0.75: logits (1, 1.25), expert 1 wins with R = 1 / (1 + e^-0.25).
    x = np.array([[1, 1, 0.5, 0.5]] * 3, dtype=np.float32)
    table = np.array([[0.0, 0.0], [0.0, 0.75]], dtype=np.float32)
    g = oracle_mod.gate_per_source(x, 0, 2, table, np.array([0, 1, 7]), want_probs=True)
    assert list(g.idx) == [0, 1, 0]                        # source 7 does not exist: no bias
    assert np.isclose(g.R[0], 1.0 / (1.0 + np.exp(-0.5))) and np.isclose(g.R[1], 1.0 / (1.0 + np.exp(-0.25)))
    assert g.R[2] == g.R[0]
    assert np.allclose(g.probs.sum(1), 1.0)
    # the cosine ignores the bias: it is the angle to the chosen expert's weight
    assert np.isclose(g.cos[0], 2.0 / (np.sqrt(2.0) * np.sqrt(2.5))) and np.isclose(g.cos[1], 1.0 / (np.sqrt(2.0) * np.sqrt(2.5)))


def test_per_source_bias_with_equal_rows_is_the_plain_bias(oracle_mod):
    rng = np.random.default_rng(3)
    x = rng.standard_normal((300, 64)).astype(np.float32)
    eps = rng.uniform(-0.1, 0.1, 8).astype(np.float32)
    src = rng.integers(0, 4, 300)
    a = oracle_mod.gate(x, 0, 8, eps=eps, want_probs=True)
    b = oracle_mod.gate_per_source(x, 0, 8, np.tile(eps, (4, 1)), src, want_probs=True)
    assert np.array_equal(a.idx, b.idx) and np.array_equal(a.R, b.R) and np.array_equal(a.cos, b.cos)
    assert np.array_equal(a.probs, b.probs)
