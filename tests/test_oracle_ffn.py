"""Pins for the oracle's expert FFN (first equation of Sec. 3.2.1: W_out . GeLU(W_in . x), GeLU = x * Phi(x))."""
import numpy as np
from scipy.stats import norm


def _bf16(a):
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    r = ((u >> 16) & 1) + 0x7FFF
    return ((u + r) >> 16).astype(np.uint16)


def _f64(bits):
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def test_ffn_matches_library_matmul_and_gaussian_cdf(oracle_mod):
    rng = np.random.default_rng(50)
    n, H, F = 5, 24, 40
    x = _bf16(rng.standard_normal((n, H)))
    w_in = _bf16(rng.standard_normal((F, H)) * 0.3)
    w_out = _bf16(rng.standard_normal((H, F)) * 0.3)
    y, spread = oracle_mod.ffn_rows(x, w_in, w_out)
    h = _f64(x) @ _f64(w_in).T
    g = h * norm.cdf(h)                       # Sec. 3.2.1 defines GeLU as the input times the standard normal CDF
    assert np.allclose(y, g @ _f64(w_out).T, rtol=1e-12, atol=1e-14)
    terms = _f64(w_out)[None, :, :] * g[:, None, :]
    assert np.allclose(spread, np.sqrt((terms ** 2).sum(-1)), rtol=1e-12)


def test_ffn_special_inputs(oracle_mod):
    # zero token -> zero output (GeLU(0) = 0); large positive pre-activation -> identity; large negative -> 0
    H, F = 8, 8
    eye = _bf16(np.eye(8) * 16.0)
    x = _bf16(np.array([[0] * 8, [1, -1, 2, -2, 0.5, -0.5, 4, -4]], np.float32))
    y, _ = oracle_mod.ffn_rows(x, eye, _bf16(np.eye(8)))
    assert not y[0].any()
    want = np.array([16, 0, 32, 0, 8, 0, 64, 0], float)       # GeLU(+16k) = 16k, GeLU(-16k) = 0 to double precision
    assert np.allclose(y[1], want, atol=1e-9)
