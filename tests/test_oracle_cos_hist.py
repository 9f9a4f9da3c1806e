"""Pins of the oracle's cosine-frequency diagnostic (Sec. 4.1, second cosine-histogram figure)."""
import numpy as np

import oracle


def _dense_weight(E, H):
    g = H // E
    W = np.zeros((E, H))
    for i in range(E):
        W[i, i * g:(i + 1) * g] = E / H
    return W


def test_against_numpy_histogram_of_dense_weight_cosines():
    rng = np.random.default_rng(11)
    T, H, E, nb = 4000, 96, 8, 40
    x = rng.standard_normal((T, H)).astype(np.float32)
    g = oracle.gate(x, oracle.F32, E)
    W = _dense_weight(E, H)
    xd = x.astype(np.float64)
    cos_all = (xd @ W.T) / (np.linalg.norm(W, axis=1)[None, :] * np.linalg.norm(xd, axis=1)[:, None])
    e, j = 3, 6
    sel = g.idx == e
    n, he, hj, ce, cj = oracle.cos_hist(x, oracle.F32, E, g.idx, e, j, nb, -0.5, 0.75)
    assert n == sel.sum() and he.sum() == n and hj.sum() == n
    assert np.allclose(ce[sel], cos_all[sel, e], rtol=0, atol=1e-14) and np.isnan(ce[~sel]).all()
    assert np.allclose(ce[sel], g.cos[sel], rtol=0, atol=1e-14)       # the routed cosine is the gate's own output
    edges = np.linspace(-0.5, 0.75, nb + 1)
    for h, c in ((he, cos_all[sel, e]), (hj, cos_all[sel, j])):
        want, _ = np.histogram(np.clip(c, -0.5, np.nextafter(0.75, 0)), bins=edges)
        near = sum(int(np.min(np.abs(v - edges)) < 1e-12) for v in c)
        assert np.abs(h - want).sum() <= 2 * near
    # routed tokens have a positive cosine to their own expert (ReLU gate: the winning mean is positive)
    assert (ce[sel] > 0).all() and cj[sel].mean() < ce[sel].mean()


def test_aligned_and_orthogonal_tokens_land_in_the_edge_bins():
    H, E, nb = 32, 4, 10
    g = H // E
    x = np.zeros((6, H), np.float32)
    x[:3, 1 * g:2 * g] = [[2.0], [0.5], [7.0]]            # multiples of w_1: cos = 1 to expert 1, 0 to expert 2
    x[3:, 0:g] = 1.0                                       # routed elsewhere
    idx = oracle.gate(x, oracle.F32, E).idx
    assert list(idx) == [1, 1, 1, 0, 0, 0]
    n, he, hj, ce, cj = oracle.cos_hist(x, oracle.F32, E, idx, 1, 2, nb, 0.0, 1.0)
    assert n == 3 and he[nb - 1] == 3 and he[:-1].sum() == 0       # cos = 1 >= hi: last bin
    assert hj[0] == 3 and hj[1:].sum() == 0                         # cos = 0 = lo: first bin
    assert np.allclose(ce[:3], 1.0, atol=1e-15) and np.all(cj[:3] == 0.0)


def test_zero_token_and_values_below_the_range():
    H, E = 8, 2
    x = np.zeros((2, H), np.float32)
    x[1, :4] = 1.0
    x[1, 4:] = -3.0
    idx = np.array([0, 0], np.int32)
    n, he, hj, ce, cj = oracle.cos_hist(x, oracle.F32, E, idx, 0, 1, 4, 0.0, 1.0)
    assert n == 2 and ce[0] == 0.0 and cj[0] == 0.0                 # |x| = 0: cosine reported as 0
    assert cj[1] < 0 and hj[0] == 2                                  # a negative cosine counts in the first bin
    want = 4.0 / (2.0 * np.sqrt(4 + 36))
    assert np.isclose(ce[1], want, rtol=1e-15)
