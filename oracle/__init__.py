"""ctypes loader for the CPU oracle (test infrastructure, not product code).

Only tests, the smoke check and the bench's CPU-baseline leg may import this
package.  It builds ``locmoe_oracle.c`` with gcc on first use and exposes thin
numpy wrappers around its functions; all arithmetic lives in the C file.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "locmoe_oracle.c")
_LIB = os.path.join(_HERE, "liblocmoe_oracle.so")

F32, BF16 = 0, 1
LAYOUT_SEND, LAYOUT_RECV = 0, 1
BOUND_BETA, BOUND_ERFC, BOUND_EXP = 0, 1, 2
WARN_CLAMPED, WARN_BAD_SRC = 1, 2


def build(force: bool = False) -> str:
    """Compile the oracle with gcc -O2 (single-threaded, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.run(
            ["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-D_DEFAULT_SOURCE", "-o", tmp, _SRC, "-lm"],
            check=True,
        )
        os.replace(tmp, _LIB)
    return _LIB


class _Rule(C.Structure):
    _fields_ = [("min_mult", C.c_double), ("capacity_factor", C.c_double),
                ("delta_override", C.c_double), ("bound_form", C.c_int32)]


class _Cap(C.Structure):
    _fields_ = [("delta", C.c_double), ("p_delta", C.c_double), ("ec_min", C.c_double),
                ("C_expert", C.c_int32), ("C_local", C.c_int32),
                ("n_empty_experts", C.c_int32), ("flags", C.c_int32)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.oracle_p_delta.restype = C.c_double
        L.oracle_p_delta.argtypes = [C.c_double, C.c_int32]
        L.oracle_ec_min.restype = C.c_double
        L.oracle_ec_min.argtypes = [C.c_double, C.c_int32, C.c_int32, C.c_int32]
        L.oracle_gate.restype = C.c_int
        L.oracle_gate.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int32, C.c_int32, C.c_void_p,
                                  C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.oracle_capacity.restype = C.c_int
        L.oracle_capacity.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int32, C.c_int32, C.c_int32,
                                      C.POINTER(_Rule), C.c_void_p, C.c_void_p, C.POINTER(_Cap)]
        L.oracle_route.restype = C.c_int
        L.oracle_route.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int32, C.c_int32, C.c_int32,
                                   C.c_int32, C.c_int32, C.c_int32] + [C.c_void_p] * 10
        L.oracle_pos_bruteforce.restype = None
        L.oracle_pos_bruteforce.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p]
        L.oracle_dest_order.restype = None
        L.oracle_dest_order.argtypes = [C.c_int32, C.c_int32, C.c_void_p]
        L.oracle_grap_weight.restype = None
        L.oracle_grap_weight.argtypes = [C.c_int32, C.c_int32, C.c_void_p]
        L.oracle_dispatch.restype = C.c_int
        L.oracle_dispatch.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int32, C.c_void_p, C.c_int64, C.c_void_p]
        L.oracle_combine.restype = C.c_int
        L.oracle_combine.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int32, C.c_void_p, C.c_void_p,
                                     C.c_void_p, C.c_void_p]
        L.oracle_ffn_rows.restype = C.c_int
        L.oracle_ffn_rows.argtypes = [C.c_void_p, C.c_int64, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p,
                                      C.c_void_p, C.c_void_p]
        L.oracle_aux_loss.restype = C.c_double
        L.oracle_aux_loss.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int32, C.c_double, C.c_void_p, C.c_void_p]
        L.oracle_loc_loss.restype = C.c_double
        L.oracle_loc_loss.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_double, C.c_double,
                                      C.c_void_p, C.c_void_p]
        L.oracle_cos_hist.restype = C.c_int64
        L.oracle_cos_hist.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int32, C.c_int32, C.c_void_p, C.c_int32, C.c_int32,
                                      C.c_int32, C.c_double, C.c_double, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.oracle_gate_topk.restype = C.c_int
        L.oracle_gate_topk.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int32, C.c_int32, C.c_void_p, C.c_int32,
                                       C.c_void_p, C.c_void_p, C.c_void_p]
        L.oracle_combine_topk.restype = C.c_int
        L.oracle_combine_topk.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p,
                                          C.c_void_p]
        _lib = L
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _raw(x, dtype):
    """Token storage as the oracle reads it: float32 array, or uint16 array of bf16 bits."""
    x = np.ascontiguousarray(x)
    if dtype == F32:
        assert x.dtype == np.float32
    else:
        assert x.dtype == np.uint16
    return x


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


@dataclass
class GateOut:
    idx: np.ndarray
    R: np.ndarray
    cos: np.ndarray
    gap: np.ndarray
    G: np.ndarray | None = None
    probs: np.ndarray | None = None


def gate(x, dtype, E, eps=None, want_G=False, want_probs=False) -> GateOut:
    x = _raw(x, dtype)
    T, H = x.shape
    idx = np.empty(T, np.int32)
    R = np.empty(T, np.float64)
    cs = np.empty(T, np.float64)
    gap = np.empty(T, np.float64)
    G = np.empty((T, E), np.float64) if want_G else None
    pr = np.empty((T, E), np.float64) if want_probs else None
    if eps is not None:
        eps = np.ascontiguousarray(eps, dtype=np.float32)
    rc = lib().oracle_gate(_p(x), dtype, T, H, E, _p(eps), _p(idx), _p(R), _p(cs), _p(gap), _p(G), _p(pr))
    if rc != 0:
        raise ValueError("oracle_gate: error %d" % rc)
    return GateOut(idx, R, cs, gap, G, pr)


def gate_per_source(x, dtype, E, eps_table, src, want_probs=False) -> GateOut:
    """The gate with a per-source-device bias table eps_table[D][E]: token t is gated with the row of its source
    device src[t] (no bias when src[t] is outside [0, D)).  The oracle's gate routine is simply called once per
    source device on that device's tokens; nothing is computed here."""
    eps_table = np.ascontiguousarray(eps_table, dtype=np.float32)
    src = np.asarray(src)
    D = eps_table.shape[0]
    T = src.shape[0]
    out = GateOut(np.empty(T, np.int32), np.empty(T, np.float64), np.empty(T, np.float64), np.empty(T, np.float64), None,
                  np.empty((T, E), np.float64) if want_probs else None)
    groups = [(np.nonzero(src == d)[0], eps_table[d]) for d in range(D)]
    groups.append((np.nonzero((src < 0) | (src >= D))[0], None))
    for sel, row in groups:
        if len(sel) == 0:
            continue
        g = gate(np.ascontiguousarray(np.asarray(x)[sel]), dtype, E, eps=row, want_probs=want_probs)
        out.idx[sel], out.R[sel], out.cos[sel], out.gap[sel] = g.idx, g.R, g.cos, g.gap
        if want_probs:
            out.probs[sel] = g.probs
    return out


def p_delta(delta: float, d: int) -> float:
    return lib().oracle_p_delta(float(delta), int(d))


def ec_min(delta: float, n: int, d: int, form: int = BOUND_BETA) -> float:
    return lib().oracle_ec_min(float(delta), int(n), int(d), int(form))


@dataclass
class CapacityOut:
    delta_e: np.ndarray
    theta_e: np.ndarray
    delta: float
    p_delta: float
    ec_min: float
    C_expert: int
    C_local: int
    n_empty_experts: int
    flags: int


def capacity(idx, cos, E, d, D, min_mult=1.0, capacity_factor=1.0, delta_override=-1.0,
             bound_form=BOUND_BETA) -> CapacityOut:
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    cos = np.ascontiguousarray(cos, dtype=np.float64)
    T = idx.shape[0]
    de = np.empty(E, np.float64)
    te = np.empty(E, np.float64)
    rule = _Rule(min_mult, capacity_factor, delta_override, bound_form)
    cap = _Cap()
    rc = lib().oracle_capacity(_p(idx), _p(cos), T, E, d, D, C.byref(rule), _p(de), _p(te), C.byref(cap))
    if rc != 0:
        raise ValueError("oracle_capacity: error %d" % rc)
    return CapacityOut(de, te, cap.delta, cap.p_delta, cap.ec_min, cap.C_expert, cap.C_local,
                       cap.n_empty_experts, cap.flags)


@dataclass
class RouteOut:
    pos: np.ndarray
    slot: np.ndarray
    drop: np.ndarray
    inv: np.ndarray
    counts: np.ndarray
    kept: np.ndarray
    send_counts: np.ndarray
    load: np.ndarray
    locality: np.ndarray
    status: int


def route(idx, src, E, N, Dn, C_local, C_alloc, layout=LAYOUT_SEND) -> RouteOut:
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    src = np.ascontiguousarray(src, dtype=np.int32)
    T = idx.shape[0]
    D = N * Dn
    pos = np.empty(T, np.int32)
    slot = np.empty(T, np.int32)
    drop = np.empty(T, np.uint8)
    inv = np.empty(D * E * C_alloc, np.int32)
    counts = np.empty((D, E), np.int32)
    kept = np.empty((D, E), np.int32)
    sc = np.empty((D, D), np.int32)
    load = np.empty(E, np.int32)
    loc = np.empty((2, 3), np.int64)
    st = np.zeros(1, np.int32)
    rc = lib().oracle_route(_p(idx), _p(src), T, E, N, Dn, C_local, C_alloc, layout, _p(pos), _p(slot),
                            _p(drop), _p(inv), _p(counts), _p(kept), _p(sc), _p(load), _p(loc), _p(st))
    if rc != 0:
        raise ValueError("oracle_route: error %d" % rc)
    return RouteOut(pos, slot, drop, inv, counts, kept, sc, load, loc, int(st[0]))


def pos_bruteforce(idx, src) -> np.ndarray:
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    src = np.ascontiguousarray(src, dtype=np.int32)
    pos = np.empty(idx.shape[0], np.int32)
    lib().oracle_pos_bruteforce(_p(idx), _p(src), idx.shape[0], _p(pos))
    return pos


def dest_order(N, Dn) -> np.ndarray:
    D = N * Dn
    r = np.empty((D, D), np.int32)
    lib().oracle_dest_order(N, Dn, _p(r))
    return r


def grap_weight(n, d) -> np.ndarray:
    w = np.empty((n, d), np.float64)
    lib().oracle_grap_weight(n, d, _p(w))
    return w


def dispatch(x, dtype, slot, rows) -> np.ndarray:
    x = _raw(x, dtype)
    T, H = x.shape
    slot = np.ascontiguousarray(slot, dtype=np.int32)
    buf = np.empty((rows, H), x.dtype)
    rc = lib().oracle_dispatch(_p(x), dtype, T, H, _p(slot), rows, _p(buf))
    if rc != 0:
        raise ValueError("oracle_dispatch: error %d" % rc)
    return buf


def combine(y, y_dtype, slot, R, prev=None) -> np.ndarray:
    y = _raw(y, y_dtype)
    H = y.shape[1]
    slot = np.ascontiguousarray(slot, dtype=np.int32)
    R = np.ascontiguousarray(R, dtype=np.float64)
    T = slot.shape[0]
    if prev is not None:
        prev = np.ascontiguousarray(prev, dtype=np.float64)
    out = np.empty((T, H), np.float64)
    rc = lib().oracle_combine(_p(y), y_dtype, T, H, _p(slot), _p(R), _p(prev), _p(out))
    if rc != 0:
        raise ValueError("oracle_combine: error %d" % rc)
    return out


def ffn_rows(x_bits, w_in_bits, w_out_bits):
    """Expert FFN of one expert on rows x [n][H]; w_in [F][H], w_out [H][F] (bf16 bits).  Returns (y, spread)."""
    x = _raw(x_bits, BF16)
    w_in = _raw(w_in_bits, BF16)
    w_out = _raw(w_out_bits, BF16)
    n, H = x.shape
    F = w_in.shape[0]
    assert w_in.shape == (F, H) and w_out.shape == (H, F)
    y = np.empty((n, H), np.float64)
    sp = np.empty((n, H), np.float64)
    rc = lib().oracle_ffn_rows(_p(x), n, H, F, _p(w_in), _p(w_out), _p(y), _p(sp))
    if rc != 0:
        raise ValueError("oracle_ffn_rows: error %d" % rc)
    return y, sp


def aux_loss(idx, probs, alpha=0.01):
    """(L_aux, f, P) of Sec. 3.2.2 from the arg-max indices and the probability matrix [T][E]."""
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    probs = np.ascontiguousarray(probs, dtype=np.float64)
    T, E = probs.shape
    f = np.empty(E, np.float64)
    P = np.empty(E, np.float64)
    L = lib().oracle_aux_loss(_p(idx), _p(probs), T, E, float(alpha), _p(f), _p(P))
    return L, f, P


def loc_loss(counts, E, n_nodes, dev_per_node, level=1, mu=1.0, smooth=1e-3):
    """(L_loc, D_c rows [G][E], KL per group [G]) of Sec. 3.2.2 under the reading stated in the C source."""
    counts = np.ascontiguousarray(counts, dtype=np.int32).reshape(n_nodes * dev_per_node, E)
    G = n_nodes if level else n_nodes * dev_per_node
    dc = np.empty((G, E), np.float64)
    kl = np.empty(G, np.float64)
    L = lib().oracle_loc_loss(_p(counts), E, n_nodes, dev_per_node, int(level), float(mu), float(smooth), _p(dc), _p(kl))
    return L, dc, kl


def cos_hist(x, dtype, E, idx, e, j, nbins, lo=-1.0, hi=1.0):
    """(n routed to e, hist of cos(x, w_e), hist of cos(x, w_j), per-token cos_e, cos_j) -- Sec. 4.1 diagnostic."""
    x = _raw(x, dtype)
    T, H = x.shape
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    he = np.empty(nbins, np.int64)
    hj = np.empty(nbins, np.int64)
    ce = np.empty(T, np.float64)
    cj = np.empty(T, np.float64)
    n = lib().oracle_cos_hist(_p(x), dtype, T, H, E, _p(idx), int(e), int(j), int(nbins), float(lo), float(hi),
                              _p(he), _p(hj), _p(ce), _p(cj))
    if n < 0:
        raise ValueError("oracle_cos_hist: bad argument")
    return n, he, hj, ce, cj


def gate_topk(x, dtype, E, K, eps=None):
    """(idx_k [K][T], R_k [K][T], gap [T]) of the top-k variant of the gate."""
    x = _raw(x, dtype)
    T, H = x.shape
    idx_k = np.empty((K, T), np.int32)
    R_k = np.empty((K, T), np.float64)
    gap = np.empty(T, np.float64)
    if eps is not None:
        eps = np.ascontiguousarray(eps, dtype=np.float32)
    rc = lib().oracle_gate_topk(_p(x), dtype, T, H, E, _p(eps), int(K), _p(idx_k), _p(R_k), _p(gap))
    if rc != 0:
        raise ValueError("oracle_gate_topk: error %d" % rc)
    return idx_k, R_k, gap


def combine_topk(y, y_dtype, slot_k, R_k) -> np.ndarray:
    y = _raw(y, y_dtype)
    H = y.shape[1]
    slot_k = np.ascontiguousarray(slot_k, dtype=np.int32)
    R_k = np.ascontiguousarray(R_k, dtype=np.float64)
    K, T = slot_k.shape
    out = np.empty((T, H), np.float64)
    rc = lib().oracle_combine_topk(_p(y), y_dtype, T, H, K, _p(slot_k), _p(R_k), _p(out))
    if rc != 0:
        raise ValueError("oracle_combine_topk: error %d" % rc)
    return out
