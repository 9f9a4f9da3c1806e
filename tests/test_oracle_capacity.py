"""Pins for the oracle's capacity stage (Lemma 3, Theorem 1, the conventional
rule ec = ceil(b_s c_f / (ep n)) of Sec. 3.2.3, and the angular deviation of
the abstract)."""
import math

import numpy as np
import pytest
from scipy.special import betainc, erf, erfc


@pytest.mark.parametrize("d", [2, 3, 4, 16, 1024, 2560, 4096, 5120])
def test_p_delta_matches_regularised_incomplete_beta(oracle_mod, d):
    # Lemma 3: p_delta = 1 - I_{delta^2}(1/2, (d-1)/2), against the library's incomplete beta.
    for z in [0.0, 0.1, 0.5, 1.0, 1.5, 2.5, 4.0, 6.0]:
        delta = min(z / math.sqrt(d), 0.999)
        ref = betainc((d - 1) / 2, 0.5, 1 - delta * delta)   # = 1 - I_{delta^2}(1/2,(d-1)/2), no cancellation
        got = oracle_mod.p_delta(delta, d)
        assert got == pytest.approx(ref, rel=2e-9, abs=1e-300)
        assert got == pytest.approx(1 - betainc(0.5, (d - 1) / 2, delta * delta), rel=1e-6, abs=1e-12)


def test_p_delta_textbook_special_cases(oracle_mod):
    # d = 3 (Archimedes' hat-box theorem): the two caps |cos| >= delta cover 1 - delta of the sphere.
    # d = 2 (circle): 1 - (2/pi) asin(delta).
    for delta in [0.0, 0.1, 0.25, 0.5, 0.9, 1.0]:
        assert oracle_mod.p_delta(delta, 3) == pytest.approx(1 - delta, abs=1e-12)
        assert oracle_mod.p_delta(delta, 2) == pytest.approx(1 - 2 / math.pi * math.asin(delta), abs=1e-9)
    assert oracle_mod.p_delta(0.0, 5120) == 1.0
    assert oracle_mod.p_delta(1.0, 5120) == 0.0


def test_p_delta_at_one_over_sqrt_d_is_about_point_three(oracle_mod):
    # Lemma 3's remark and Appendix A.2: delta = sqrt(1/(d - 3/2)) gives I ~ erf(sqrt(2)/2) ~ 0.68, p ~ 0.3.
    for d in [1024, 5120]:
        p = oracle_mod.p_delta(math.sqrt(1 / (d - 1.5)), d)
        assert 1 - p == pytest.approx(erf(math.sqrt(2) / 2), abs=2e-4)
        assert round(1 - p, 2) == 0.68
        assert round(p, 1) == 0.3


def test_p_delta_monte_carlo(oracle_mod):
    # Assumption 2 + Lemma 3: share of uniform unit vectors whose |cos| to a fixed unit weight is >= delta.
    rng = np.random.default_rng(10)
    d, n_samp = 256, 200000
    x = rng.standard_normal((n_samp, d))
    c = np.abs(x[:, 0]) / np.linalg.norm(x, axis=1)
    for delta in [0.03, 1 / 16, 0.12]:
        p = oracle_mod.p_delta(delta, d)
        frac = (c >= delta).mean()
        assert abs(frac - p) < 5 * math.sqrt(p * (1 - p) / n_samp)


def test_ec_min_forms_at_the_papers_delta(oracle_mod):
    # Theorem 1 evaluated where the paper reads delta off its histogram (about 0.03, 16 experts),
    # with d = 5120: exact = 1/(n p_delta); erfc form; exp form.  Expected values from library functions.
    delta, n, d = 0.03, 16, 5120
    a = delta * delta * d / (2 - delta * delta)
    exact = 1 / (n * betainc((d - 1) / 2, 0.5, 1 - delta * delta))
    assert oracle_mod.ec_min(delta, n, d, 0) == pytest.approx(exact, rel=1e-9)
    assert oracle_mod.ec_min(delta, n, d, 1) == pytest.approx(1 / (n * erfc(math.sqrt(a))), rel=1e-13)
    assert oracle_mod.ec_min(delta, n, d, 2) == pytest.approx(math.exp(a) / n, rel=1e-13)
    # the three numbers themselves (about two tokens per expert)
    assert oracle_mod.ec_min(delta, n, d, 0) == pytest.approx(1.96481, abs=1e-5)
    assert oracle_mod.ec_min(delta, n, d, 1) == pytest.approx(1.96636, abs=1e-5)
    assert oracle_mod.ec_min(delta, n, d, 2) == pytest.approx(0.62653, abs=1e-5)


def test_ec_min_chain_and_monotonicity(oracle_mod):
    # Theorem 1's large-d chain: exact ~ erfc form > exp form (equal at delta = 0), and the bound
    # grows as the angle shrinks (delta grows).
    for d, n in [(1024, 8), (5120, 64)]:
        prev = 0.0
        for z in np.linspace(0.0, 6.0, 25):
            delta = z / math.sqrt(d)
            ex, ef, xp = (oracle_mod.ec_min(delta, n, d, f) for f in (0, 1, 2))
            assert ex == pytest.approx(ef, rel=0.03)
            assert ef >= xp * (1 - 1e-12)
            assert ex > prev
            prev = ex
        assert oracle_mod.ec_min(0.0, n, d, 0) == pytest.approx(1 / n)
        assert oracle_mod.ec_min(0.0, n, d, 1) == pytest.approx(1 / n)
        assert oracle_mod.ec_min(0.0, n, d, 2) == pytest.approx(1 / n)


def test_delta_is_the_largest_angle_per_expert(oracle_mod):
    # delta_e = smallest cosine among the tokens routed to e; theta_e = acos; delta = min_e clamped at 0.
    rng = np.random.default_rng(11)
    T, E = 1000, 8
    idx = rng.integers(0, E - 1, T).astype(np.int32)     # expert 7 stays empty
    cos = rng.uniform(0.01, 0.2, T)
    cap = oracle_mod.capacity(idx, cos, E, 1024, 8)
    for e in range(E - 1):
        assert cap.delta_e[e] == cos[idx == e].min()
        assert cap.theta_e[e] == pytest.approx(math.acos(cos[idx == e].min()), rel=1e-15)
    assert cap.delta_e[E - 1] == 1.0 and cap.theta_e[E - 1] == 0.0 and cap.n_empty_experts == 1
    assert cap.delta == cos.min()
    assert cap.p_delta == pytest.approx(betainc((1024 - 1) / 2, 0.5, 1 - cos.min() ** 2), rel=2e-9)
    cos[3] = -0.5
    assert oracle_mod.capacity(idx, cos, E, 1024, 8).delta == 0.0
    assert oracle_mod.capacity(idx, cos, E, 1024, 8, delta_override=0.03).delta == 0.03


def test_integer_capacity_rule(oracle_mod):
    # Conventional term: ec = ceil(b_s c_f / (ep n)) with b_s = T, ep = D.  Minimum term: ceil of Theorem 1.
    idx = np.zeros(65536, np.int32)
    cos = np.full(65536, 0.5)
    # config-2 shape; the minimum (about 0.02 tokens at delta = 0) never binds
    for cf, cl, ce in [(1.0, 16, 1024), (1.25, 20, 1280), (2.0, 32, 2048)]:
        cap = oracle_mod.capacity(idx, cos, 64, 5120, 64, min_mult=cf, capacity_factor=cf, delta_override=0.0)
        assert (cap.C_local, cap.C_expert) == (cl, ce)
        assert cap.ec_min == pytest.approx(1 / 64)
    # literal-minimum mode: c_f = 0, capacity = ceil(ec_min) = 1 slot
    cap = oracle_mod.capacity(idx, cos, 64, 5120, 64, capacity_factor=0.0, delta_override=0.0)
    assert (cap.C_local, cap.C_expert) == (1, 1)
    # non-divisible: T = 1000, n = 8, D = 4, c_f = 1.1 -> ceil(137.5) = 138, ceil(34.375) = 35
    cap = oracle_mod.capacity(idx[:1000], cos[:1000], 8, 1024, 4, capacity_factor=1.1, delta_override=0.0)
    assert (cap.C_expert, cap.C_local) == (138, 35)
    # the minimum binds: d = 1024, n = 8, delta = 0.1 -> ec_min ~ 1/(8 p); capacity = ceil(min_mult ec_min)
    ec = 1 / (8 * betainc((1024 - 1) / 2, 0.5, 1 - 0.01))
    cap = oracle_mod.capacity(idx[:8192], cos[:8192], 8, 1024, 8, min_mult=2.0, capacity_factor=0.01,
                              delta_override=0.1)
    assert cap.C_expert == math.ceil(2.0 * ec) and cap.C_local == math.ceil(math.ceil(2.0 * ec) / 8)
    assert cap.C_expert >= min(cap.ec_min, 8192)
    # the bound saturates at T when p_delta underflows
    cap = oracle_mod.capacity(idx[:8192], cos[:8192], 8, 1024, 8, delta_override=0.9)
    assert cap.C_expert == 8192 and cap.C_local == 1024


def test_printed_constants_of_the_paper(oracle_mod):
    import os
    vals = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", "paper_constants.txt")) as f:
        for line in f:
            line = line.split("#")[0].split()
            if len(line) == 3:
                vals[line[0]] = (float(line[1]), float(line[2]))
    for d in [1024, 2560, 5120]:
        p = oracle_mod.p_delta(math.sqrt(1 / (d - 1.5)), d)
        v, tol = vals["p_delta_at_inv_sqrt_d"]
        assert abs(p - v) <= tol
        v, tol = vals["erf_sqrt2_over_2"]
        assert abs((1 - p) - v) <= tol
    # at the paper's delta with its 16 experts the bound is a handful of tokens, far below T/n
    delta = vals["observed_delta"][0]
    assert 1.0 < oracle_mod.ec_min(delta, 16, 5120, 0) < 3.0
