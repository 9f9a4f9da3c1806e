"""Pins of the oracle's locality loss (Sec. 3.2.2, second loss equation).  The arithmetic is pinned here; whether
the paper means these two distributions is a reading (the paper gives no symbols for them)."""
import numpy as np
import pytest
from scipy.special import rel_entr

import oracle


def _local_mask(E, G):
    Eg = E // G
    return (np.arange(E)[None, :] // Eg) == np.arange(G)[:, None]


@pytest.mark.parametrize("level", [0, 1])
def test_fully_local_uniform_assignment_has_the_closed_form(level):
    # every token on a local expert, uniformly: c_s = 1 / Eg on the local experts, so
    # KL_s = ln((1 / Eg) / ((1 - l) / Eg + l / E)) = -ln(1 - l + l Eg / E) for every group
    E, N, Dn, lam = 32, 2, 4, 0.05
    D = N * Dn
    G = N if level else D
    Eg = E // G
    counts = np.zeros((D, E), np.int32)
    for d in range(D):
        s = d // Dn if level else d
        counts[d, s * Eg:(s + 1) * Eg] = 3
    L, dc, kl = oracle.loc_loss(counts, E, N, Dn, level=level, mu=2.0, smooth=lam)
    want = -np.log(1.0 - lam + lam * Eg / E)
    assert np.allclose(kl, want, rtol=1e-13)
    assert np.isclose(L, 2.0 * want, rtol=1e-13)
    assert np.allclose(dc[_local_mask(E, G)], 1.0 / Eg)


def test_zero_when_the_batch_matches_the_localised_distribution():
    # counts proportional to q_s(e): the divergence vanishes (Gibbs' inequality is tight only there)
    E, N, Dn, lam = 8, 2, 2, 0.5
    D, Eg = 4, 2
    counts = np.zeros((D, E), np.int32)
    for d in range(D):
        q = np.full(E, lam / E)
        q[d * Eg:(d + 1) * Eg] += (1 - lam) / Eg
        counts[d] = np.round(q * 1600).astype(np.int32)     # 1600 q is an integer for these numbers
    L, _, kl = oracle.loc_loss(counts, E, N, Dn, level=0, mu=1.0, smooth=lam)
    assert np.all(np.abs(kl) < 1e-14) and abs(L) < 1e-14


@pytest.mark.parametrize("level", [0, 1])
def test_against_a_library_relative_entropy_on_random_counts(level):
    rng = np.random.default_rng(5)
    E, N, Dn, lam, mu = 64, 4, 2, 1e-3, 0.7
    D = N * Dn
    G = N if level else D
    counts = rng.integers(0, 50, size=(D, E)).astype(np.int32)
    counts[rng.random((D, E)) < 0.3] = 0                    # zero cells: 0 ln 0 = 0
    counts[3] = 0                                           # a device without tokens
    L, dc, kl = oracle.loc_loss(counts, E, N, Dn, level=level, mu=mu, smooth=lam)
    grouped = counts.reshape(G, D // G, E).sum(1).astype(np.float64)
    n = grouped.sum(1)
    q = np.where(_local_mask(E, G), (1 - lam) / (E // G), 0.0) + lam / E
    joint_c = grouped / grouped.sum()
    joint_l = (n / n.sum())[:, None] * q
    assert np.isclose(L, mu * rel_entr(joint_c, joint_l).sum(), rtol=1e-12)
    assert np.all(kl >= 0.0)
    rows = n > 0
    assert np.allclose(dc[rows].sum(1), 1.0, rtol=1e-14)
    assert np.allclose(kl[rows], rel_entr(grouped[rows] / n[rows, None], q[rows]).sum(1), rtol=1e-12)


def test_everything_remote_is_the_largest_value():
    # all tokens of every device on one remote expert: KL_s = ln(1 / (l / E)) = ln(E / l)
    E, N, Dn, lam = 16, 2, 2, 1e-2
    D, Eg = 4, 4
    counts = np.zeros((D, E), np.int32)
    for d in range(D):
        counts[d, ((d + 1) % D) * Eg] = 9
    L, _, kl = oracle.loc_loss(counts, E, N, Dn, level=0, mu=1.0, smooth=lam)
    assert np.allclose(kl, np.log(E / lam), rtol=1e-13) and np.isclose(L, np.log(E / lam), rtol=1e-13)


def test_no_tokens_at_all():
    L, dc, kl = oracle.loc_loss(np.zeros((4, 8), np.int32), 8, 2, 2, level=1)
    assert L == 0.0 and not dc.any() and not kl.any()
