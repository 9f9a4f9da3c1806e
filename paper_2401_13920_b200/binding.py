"""Python face of the C-ABI library declared in ``include/locmoe.h``.

Argument marshalling only: every function hands device pointers of torch
tensors to the entry point of the same name in ``liblocmoe.so``; all of the
router's arithmetic runs in the CUDA kernels.  There is no CPU fallback -- if
the library is missing it is built with nvcc, and if that fails the import of
this module raises.
"""
from __future__ import annotations

import ctypes as C
from dataclasses import dataclass

import torch

from . import build as _build

F32, BF16 = 0, 1
LAYOUT_SEND, LAYOUT_RECV = 0, 1
BOUND_BETA, BOUND_ERFC, BOUND_EXP = 0, 1, 2
ROUTE_EARLY_INIT = 1
WARN_CLAMPED, WARN_BAD_SRC, WARN_BAD_IDX = 1, 2, 4
FLAG_DELTA_OVERRIDE, FLAG_MIN_SATURATED, FLAG_MIN_BINDS = 1, 2, 4

EXPORTS = [
    "locmoe_workspace_bytes", "locmoe_gate", "locmoe_gate_ex", "locmoe_aux_loss_partial", "locmoe_capacity", "locmoe_capacity_noalloc", "locmoe_capacity_read", "locmoe_route", "locmoe_capacity_route", "locmoe_gate_route",
    "locmoe_conventional_capacity", "locmoe_batch_delta", "locmoe_dest_order",
    "locmoe_dispatch", "locmoe_combine", "locmoe_dispatch_peer", "locmoe_dispatch_peer_window", "locmoe_combine_peer", "locmoe_topk_select", "locmoe_topk_fold", "locmoe_combine_topk", "locmoe_expert_ffn", "locmoe_ffn_kernels", "locmoe_moe_layer", "locmoe_aux_loss", "locmoe_loc_loss", "locmoe_cos_hist", "locmoe_launch_counts", "locmoe_device_flags", "locmoe_status_string",
]


class Shape(C.Structure):
    _fields_ = [("T", C.c_int32), ("H", C.c_int32), ("E", C.c_int32), ("n_nodes", C.c_int32),
                ("dev_per_node", C.c_int32), ("x_dtype", C.c_int32), ("layout", C.c_int32)]

    @property
    def D(self) -> int:
        return self.n_nodes * self.dev_per_node


class CapacityRule(C.Structure):
    _fields_ = [("min_mult", C.c_double), ("capacity_factor", C.c_double), ("delta_override", C.c_double),
                ("bound_form", C.c_int32), ("T_global", C.c_int32)]


class Capacity(C.Structure):
    _fields_ = [("delta", C.c_double), ("p_delta", C.c_double), ("ec_min", C.c_double),
                ("C_expert", C.c_int32), ("C_local", C.c_int32), ("n_empty_experts", C.c_int32),
                ("flags", C.c_int32)]


GATE_PARTIAL_ROWS = 2048


class GateOpts(C.Structure):
    _fields_ = [("eps", C.c_void_p), ("src_dev", C.c_void_p), ("probs", C.c_void_p), ("p_part", C.c_void_p),
                ("p_rows", C.c_int32)]


class LayerBuffers(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("idx", "gate_w", "cos_sim", "delta_e", "theta_e", "cap_dev", "pos", "slot",
                                           "drop", "inv", "counts", "kept", "send_counts", "load", "locality",
                                           "status", "ws")] + [("ws_bytes", C.c_size_t)] + \
               [(n, C.c_void_p) for n in ("buf", "h1", "y")]


CAPACITY_BYTES = C.sizeof(Capacity)


class LocMoEError(RuntimeError):
    def __init__(self, fn: str, code: int):
        self.code = code
        super().__init__("%s failed: %d (%s)" % (fn, code, status_string(code)))


def _load() -> C.CDLL:
    path = _build.build()  # raises when nvcc or the sources are missing
    lib = C.CDLL(path)
    vp, i32 = C.c_void_p, C.c_int32
    lib.locmoe_workspace_bytes.argtypes = [C.POINTER(Shape), i32, C.POINTER(C.c_size_t)]
    lib.locmoe_gate.argtypes = [C.POINTER(Shape), vp, vp, vp, vp, vp, vp, vp]
    lib.locmoe_gate_ex.argtypes = [C.POINTER(Shape), vp, C.POINTER(GateOpts), vp, vp, vp, vp]
    lib.locmoe_aux_loss_partial.argtypes = [C.POINTER(Shape), vp, i32, vp, C.c_float, vp, vp, vp, vp]
    lib.locmoe_capacity.argtypes = [C.POINTER(Shape), vp, vp, C.POINTER(CapacityRule), vp, vp, vp, vp, C.c_size_t, vp]
    lib.locmoe_capacity_noalloc.argtypes = [C.POINTER(Shape), vp, vp, C.POINTER(CapacityRule), vp, vp, vp, vp]
    lib.locmoe_capacity_read.argtypes = [vp, C.POINTER(Capacity), vp]
    lib.locmoe_route.argtypes = [C.POINTER(Shape), vp, vp, vp, i32] + [vp] * 10 + [vp, C.c_size_t, vp]
    lib.locmoe_capacity_route.argtypes = [C.POINTER(Shape), vp, vp, vp, C.POINTER(CapacityRule), vp, vp, vp, i32] + [vp] * 10 + \
                                         [i32, vp, C.c_size_t, vp]
    lib.locmoe_gate_route.argtypes = [C.POINTER(Shape), vp, vp, vp, C.POINTER(CapacityRule)] + [vp] * 6 + [i32] + [vp] * 10 + \
                                     [i32, vp, C.c_size_t, vp]
    lib.locmoe_dispatch.argtypes = [C.POINTER(Shape), i32, vp, vp, vp, vp, i32, vp]
    lib.locmoe_combine.argtypes = [C.POINTER(Shape), i32, vp, i32, vp, vp, vp, i32, vp]
    lib.locmoe_expert_ffn.argtypes = [C.POINTER(Shape), i32, i32, vp, vp, vp, vp, vp, i32, vp]
    lib.locmoe_ffn_kernels.argtypes = [C.POINTER(Shape), i32, i32, C.POINTER(i32 * 2)]
    lib.locmoe_moe_layer.argtypes = [C.POINTER(Shape), vp, vp, vp, C.POINTER(CapacityRule), i32, i32, vp, vp,
                                     C.POINTER(LayerBuffers), vp, vp]
    lib.locmoe_aux_loss.argtypes = [C.POINTER(Shape), vp, vp, C.c_float, vp, vp, vp, vp, C.c_size_t, vp]
    lib.locmoe_loc_loss.argtypes = [C.POINTER(Shape), vp, i32, C.c_double, C.c_double, vp, vp, vp, vp, vp]
    lib.locmoe_cos_hist.argtypes = [C.POINTER(Shape), vp, vp, i32, i32, i32, C.c_float, C.c_float, vp, vp, vp, vp]
    lib.locmoe_dispatch_peer.argtypes = [C.POINTER(Shape), i32, vp, vp, vp, C.POINTER(vp), i32, i32, i32, i32, vp]
    lib.locmoe_dispatch_peer_window.argtypes = [C.POINTER(Shape), i32, vp, vp, vp, C.POINTER(vp), i32, i32, i32, i32,
                                                C.c_int64, C.c_int64, vp]
    lib.locmoe_combine_peer.argtypes = [C.POINTER(Shape), i32, C.POINTER(vp), i32, i32, vp, vp, vp, vp]
    lib.locmoe_topk_select.argtypes = [C.POINTER(Shape), vp, vp, vp, i32, vp, vp, vp]
    lib.locmoe_topk_fold.argtypes = [C.POINTER(Shape), i32, vp, vp]
    lib.locmoe_combine_topk.argtypes = [C.POINTER(Shape), i32, vp, i32, i32, vp, vp, vp, vp]
    lib.locmoe_conventional_capacity.argtypes = [C.POINTER(Shape), C.POINTER(CapacityRule), C.POINTER(C.c_int32)]
    lib.locmoe_batch_delta.argtypes = [vp, i32, C.POINTER(C.c_double)]
    lib.locmoe_dest_order.argtypes = [C.POINTER(Shape), i32, i32]
    lib.locmoe_launch_counts.argtypes = [C.POINTER(Shape), C.POINTER(C.c_int32 * 5)]
    lib.locmoe_device_flags.argtypes = [C.POINTER(C.c_int32), vp]
    lib.locmoe_status_string.argtypes = [C.c_int]
    lib.locmoe_status_string.restype = C.c_char_p
    for name in EXPORTS[:-1]:
        getattr(lib, name).restype = C.c_int
    return lib


_lib = _load()


def library_path() -> str:
    return _build.LIB


def status_string(code: int) -> str:
    return _lib.locmoe_status_string(int(code)).decode()


def dtype_code(dt: torch.dtype) -> int:
    if dt == torch.float32:
        return F32
    if dt == torch.bfloat16:
        return BF16
    raise TypeError("tokens must be float32 or bfloat16, got %s" % dt)


def make_shape(T, H, E, n_nodes, dev_per_node, x_dtype, layout=LAYOUT_SEND) -> Shape:
    if isinstance(x_dtype, torch.dtype):
        x_dtype = dtype_code(x_dtype)
    return Shape(int(T), int(H), int(E), int(n_nodes), int(dev_per_node), int(x_dtype), int(layout))


def _ptr(t):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("expected a CUDA tensor")
    if not t.is_contiguous():
        raise ValueError("expected a contiguous tensor")
    return C.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def _check(fn: str, rc: int) -> int:
    if rc < 0:
        raise LocMoEError(fn, rc)
    return rc


def _want(t, dtype, numel, name):
    if t.dtype != dtype or t.numel() < numel:
        raise ValueError("%s: expected %s with at least %d elements, got %s with %d"
                         % (name, dtype, numel, t.dtype, t.numel()))


def locmoe_workspace_bytes(shape: Shape, C_alloc: int) -> int:
    out = C.c_size_t(0)
    _check("locmoe_workspace_bytes", _lib.locmoe_workspace_bytes(C.byref(shape), int(C_alloc), C.byref(out)))
    return out.value


def locmoe_launch_counts(shape: Shape) -> dict:
    out = (C.c_int32 * 5)()
    _check("locmoe_launch_counts", _lib.locmoe_launch_counts(C.byref(shape), C.byref(out)))
    return dict(zip(("gate", "capacity", "route", "dispatch", "combine"), list(out)))


def locmoe_device_flags(stream=None) -> int:
    out = C.c_int32(0)
    _check("locmoe_device_flags", _lib.locmoe_device_flags(C.byref(out), _stream(stream)))
    return out.value


def locmoe_gate(shape: Shape, x, eps, idx, gate_w, cos_sim, probs=None, stream=None) -> int:
    _want(x, torch.float32 if shape.x_dtype == F32 else torch.bfloat16, shape.T * shape.H, "x")
    _want(idx, torch.int32, shape.T, "idx")
    _want(gate_w, torch.float32, shape.T, "gate_w")
    _want(cos_sim, torch.float32, shape.T, "cos_sim")
    if eps is not None:
        _want(eps, torch.float32, shape.E, "eps")
    if probs is not None:
        _want(probs, torch.float32, shape.T * shape.E, "probs")
    return _check("locmoe_gate", _lib.locmoe_gate(C.byref(shape), _ptr(x), _ptr(eps), _ptr(idx), _ptr(gate_w),
                                                  _ptr(cos_sim), _ptr(probs), _stream(stream)))


def locmoe_gate_ex(shape: Shape, x, idx, gate_w, cos_sim, eps=None, src_dev=None, probs=None, p_part=None, stream=None) -> int:
    """The gate with its extras; returns the number of rows of ``p_part`` the call wrote (0 without ``p_part``).
    ``eps`` is float[E], or float[D][E] when ``src_dev`` (int32[T]) is given: the per-source bias table."""
    _want(x, torch.float32 if shape.x_dtype == F32 else torch.bfloat16, shape.T * shape.H, "x")
    _want(idx, torch.int32, shape.T, "idx")
    _want(gate_w, torch.float32, shape.T, "gate_w")
    _want(cos_sim, torch.float32, shape.T, "cos_sim")
    if eps is not None:
        _want(eps, torch.float32, shape.E * (shape.D if src_dev is not None else 1), "eps")
    if src_dev is not None:
        _want(src_dev, torch.int32, shape.T, "src_dev")
    if probs is not None:
        _want(probs, torch.float32, shape.T * shape.E, "probs")
    if p_part is not None:
        _want(p_part, torch.float32, GATE_PARTIAL_ROWS * shape.E, "p_part")
    p = lambda t: None if t is None else _ptr(t).value
    opts = GateOpts(p(eps), p(src_dev), p(probs), p(p_part), 0)
    _check("locmoe_gate_ex", _lib.locmoe_gate_ex(C.byref(shape), _ptr(x), C.byref(opts), _ptr(idx), _ptr(gate_w), _ptr(cos_sim),
                                                 _stream(stream)))
    return opts.p_rows


def locmoe_aux_loss_partial(shape: Shape, p_part, p_rows, load, alpha, f_out, p_out, loss_out, stream=None) -> int:
    _want(p_part, torch.float32, p_rows * shape.E, "p_part")
    _want(load, torch.int32, shape.E, "load")
    _want(f_out, torch.float32, shape.E, "f_out")
    _want(p_out, torch.float32, shape.E, "p_out")
    _want(loss_out, torch.float32, 1, "loss_out")
    return _check("locmoe_aux_loss_partial", _lib.locmoe_aux_loss_partial(C.byref(shape), _ptr(p_part), int(p_rows), _ptr(load),
                                                                          float(alpha), _ptr(f_out), _ptr(p_out), _ptr(loss_out),
                                                                          _stream(stream)))


def locmoe_capacity(shape: Shape, idx, cos_sim, rule: CapacityRule, delta_e, theta_e, cap_dev, ws, stream=None) -> int:
    _want(idx, torch.int32, shape.T, "idx")
    _want(cos_sim, torch.float32, shape.T, "cos_sim")
    _want(delta_e, torch.float32, shape.E, "delta_e")
    _want(theta_e, torch.float32, shape.E, "theta_e")
    _want(cap_dev, torch.uint8, CAPACITY_BYTES, "cap_dev")
    return _check("locmoe_capacity", _lib.locmoe_capacity(
        C.byref(shape), _ptr(idx), _ptr(cos_sim), C.byref(rule), _ptr(delta_e), _ptr(theta_e), _ptr(cap_dev),
        _ptr(ws), ws.numel() * ws.element_size(), _stream(stream)))


def locmoe_capacity_noalloc(shape: Shape, idx, cos_sim, rule: CapacityRule, delta_e, theta_e, cap_dev, stream=None) -> int:
    """locmoe_capacity without a workspace argument: for callers that cannot allocate device memory (the
    scratch is a fixed array inside the library, at most 8192 experts, shared by all calls on a device)."""
    _want(idx, torch.int32, shape.T, "idx")
    _want(cos_sim, torch.float32, shape.T, "cos_sim")
    _want(delta_e, torch.float32, shape.E, "delta_e")
    _want(theta_e, torch.float32, shape.E, "theta_e")
    _want(cap_dev, torch.uint8, CAPACITY_BYTES, "cap_dev")
    return _check("locmoe_capacity_noalloc", _lib.locmoe_capacity_noalloc(
        C.byref(shape), _ptr(idx), _ptr(cos_sim), C.byref(rule), _ptr(delta_e), _ptr(theta_e), _ptr(cap_dev),
        _stream(stream)))


def locmoe_capacity_read(cap_dev, stream=None) -> Capacity:
    out = Capacity()
    _check("locmoe_capacity_read", _lib.locmoe_capacity_read(_ptr(cap_dev), C.byref(out), _stream(stream)))
    return out


def locmoe_route(shape: Shape, idx, src_dev, cap_dev, C_alloc, pos, slot, drop, inv, counts, kept, send_counts,
                 load, locality, status, ws, stream=None) -> int:
    D, E, T = shape.D, shape.E, shape.T
    _want(idx, torch.int32, T, "idx")
    _want(src_dev, torch.int32, T, "src_dev")
    _want(cap_dev, torch.uint8, CAPACITY_BYTES, "cap_dev")
    _want(pos, torch.int32, T, "pos")
    _want(slot, torch.int32, T, "slot")
    _want(drop, torch.uint8, T, "drop")
    _want(inv, torch.int32, D * E * C_alloc, "inv")
    _want(counts, torch.int32, D * E, "counts")
    _want(kept, torch.int32, D * E, "kept")
    _want(send_counts, torch.int32, D * D, "send_counts")
    _want(load, torch.int32, E, "load")
    _want(locality, torch.int64, 6, "locality")
    _want(status, torch.int32, 1, "status")
    return _check("locmoe_route", _lib.locmoe_route(
        C.byref(shape), _ptr(idx), _ptr(src_dev), _ptr(cap_dev), int(C_alloc), _ptr(pos), _ptr(slot), _ptr(drop),
        _ptr(inv), _ptr(counts), _ptr(kept), _ptr(send_counts), _ptr(load), _ptr(locality), _ptr(status),
        _ptr(ws), ws.numel() * ws.element_size(), _stream(stream)))


def locmoe_capacity_route(shape: Shape, idx, cos_sim, src_dev, rule: CapacityRule, delta_e, theta_e, cap_dev, C_alloc, pos, slot,
                          drop, inv, counts, kept, send_counts, load, locality, status, ws, stream=None, early_init=False) -> int:
    D, E, T = shape.D, shape.E, shape.T
    for t, dt, n, name in ((idx, torch.int32, T, "idx"), (cos_sim, torch.float32, T, "cos_sim"), (src_dev, torch.int32, T, "src_dev"),
                           (delta_e, torch.float32, E, "delta_e"), (theta_e, torch.float32, E, "theta_e"),
                           (cap_dev, torch.uint8, CAPACITY_BYTES, "cap_dev"), (pos, torch.int32, T, "pos"),
                           (slot, torch.int32, T, "slot"), (drop, torch.uint8, T, "drop"), (inv, torch.int32, D * E * C_alloc, "inv"),
                           (counts, torch.int32, D * E, "counts"), (kept, torch.int32, D * E, "kept"),
                           (send_counts, torch.int32, D * D, "send_counts"), (load, torch.int32, E, "load"),
                           (locality, torch.int64, 6, "locality"), (status, torch.int32, 1, "status")):
        _want(t, dt, n, name)
    return _check("locmoe_capacity_route", _lib.locmoe_capacity_route(
        C.byref(shape), _ptr(idx), _ptr(cos_sim), _ptr(src_dev), C.byref(rule), _ptr(delta_e), _ptr(theta_e), _ptr(cap_dev),
        int(C_alloc), _ptr(pos), _ptr(slot), _ptr(drop), _ptr(inv), _ptr(counts), _ptr(kept), _ptr(send_counts), _ptr(load),
        _ptr(locality), _ptr(status), ROUTE_EARLY_INIT if early_init else 0, _ptr(ws), ws.numel() * ws.element_size(),
        _stream(stream)))


def locmoe_gate_route(shape: Shape, x, eps, src_dev, rule: CapacityRule, st: "RouterState", stream=None, early_init=False) -> int:
    """Gate, capacity and route as one call chain on the tensors of a RouterState."""
    dt = torch.float32 if shape.x_dtype == F32 else torch.bfloat16
    _want(x, dt, shape.T * shape.H, "x")
    _want(src_dev, torch.int32, shape.T, "src_dev")
    if eps is not None:
        _want(eps, torch.float32, shape.E, "eps")
    return _check("locmoe_gate_route", _lib.locmoe_gate_route(
        C.byref(shape), _ptr(x), _ptr(eps), _ptr(src_dev), C.byref(rule), _ptr(st.idx), _ptr(st.gate_w), _ptr(st.cos_sim),
        _ptr(st.delta_e), _ptr(st.theta_e), _ptr(st.cap_dev), int(st.C_alloc), _ptr(st.pos), _ptr(st.slot), _ptr(st.drop),
        _ptr(st.inv), _ptr(st.counts), _ptr(st.kept), _ptr(st.send_counts), _ptr(st.load), _ptr(st.locality), _ptr(st.status),
        ROUTE_EARLY_INIT if early_init else 0, _ptr(st.ws), st.ws.numel() * st.ws.element_size(), _stream(stream)))


def locmoe_dispatch(shape: Shape, C_alloc, x, inv, buf, zero_pad=True, stream=None, slot=None) -> int:
    rows = shape.D * shape.E * C_alloc
    dt = torch.float32 if shape.x_dtype == F32 else torch.bfloat16
    _want(x, dt, shape.T * shape.H, "x")
    _want(inv, torch.int32, rows, "inv")
    _want(buf, dt, rows * shape.H, "buf")
    if slot is not None:
        _want(slot, torch.int32, shape.T, "slot")
    return _check("locmoe_dispatch", _lib.locmoe_dispatch(C.byref(shape), int(C_alloc), _ptr(x), _ptr(inv), _ptr(slot),
                                                          _ptr(buf), 1 if zero_pad else 0, _stream(stream)))


def locmoe_combine(shape: Shape, C_alloc, y, slot, gate_w, out, accumulate=False, stream=None) -> int:
    rows = shape.D * shape.E * C_alloc
    _want(y, y.dtype, rows * shape.H, "y")
    _want(slot, torch.int32, shape.T, "slot")
    _want(gate_w, torch.float32, shape.T, "gate_w")
    _want(out, torch.float32 if shape.x_dtype == F32 else torch.bfloat16, shape.T * shape.H, "out")
    return _check("locmoe_combine", _lib.locmoe_combine(C.byref(shape), int(C_alloc), _ptr(y), dtype_code(y.dtype),
                                                        _ptr(slot), _ptr(gate_w), _ptr(out), 1 if accumulate else 0,
                                                        _stream(stream)))


FFN_KERNEL_NAMES = ("ffn_gemm_kernel (128 x 256 tiles)", "ffn_gemm_wide_kernel (256 x 256 tiles)",
                    "ffn_gemm2_kernel (two SMs per tile)", "ffn_gemm2_kernel (two SMs per tile, one accumulator)")


def locmoe_ffn_kernels(shape: Shape, C_alloc, F):
    """Which kernel the library runs each of the two GEMMs of locmoe_expert_ffn with (host only): two codes."""
    out = (C.c_int32 * 2)()
    _check("locmoe_ffn_kernels", _lib.locmoe_ffn_kernels(C.byref(shape), int(C_alloc), int(F), C.byref(out)))
    return int(out[0]), int(out[1])


def locmoe_expert_ffn(shape: Shape, C_alloc, F, buf, w_in, w_out, h1, y, stream=None) -> int:
    rows = shape.D * shape.E * C_alloc
    _want(buf, torch.bfloat16, rows * shape.H, "buf")
    _want(w_in, torch.bfloat16, shape.E * F * shape.H, "w_in")
    _want(w_out, torch.bfloat16, shape.E * shape.H * F, "w_out")
    _want(h1, torch.bfloat16, rows * F, "h1")
    _want(y, y.dtype, rows * shape.H, "y")
    return _check("locmoe_expert_ffn", _lib.locmoe_expert_ffn(C.byref(shape), int(C_alloc), int(F), _ptr(buf), _ptr(w_in),
                                                              _ptr(w_out), _ptr(h1), _ptr(y), dtype_code(y.dtype),
                                                              _stream(stream)))


def locmoe_aux_loss(shape: Shape, probs, load, alpha, f_out, p_out, loss_out, ws, stream=None) -> int:
    _want(probs, torch.float32, shape.T * shape.E, "probs")
    _want(load, torch.int32, shape.E, "load")
    _want(f_out, torch.float32, shape.E, "f_out")
    _want(p_out, torch.float32, shape.E, "p_out")
    _want(loss_out, torch.float32, 1, "loss_out")
    return _check("locmoe_aux_loss", _lib.locmoe_aux_loss(C.byref(shape), _ptr(probs), _ptr(load), float(alpha),
                                                          _ptr(f_out), _ptr(p_out), _ptr(loss_out), _ptr(ws),
                                                          ws.numel() * ws.element_size(), _stream(stream)))


def _ptr_table(ptrs):
    """Host array of device pointers (ints or CUDA tensors) for the peer calls."""
    vals = [p.data_ptr() if hasattr(p, "data_ptr") else int(p) for p in ptrs]
    return (C.c_void_p * len(vals))(*vals), len(vals)


def locmoe_dispatch_peer(shape: Shape, C_alloc, x, inv, slot, peer_bufs, src_lo, src_hi, zero_pad=True, stream=None,
                         window=None) -> int:
    """``window`` = (lo, hi): only rows whose index inside their owner's slice lies in [lo, hi) (locmoe_dispatch_peer_window)."""
    rows = shape.D * shape.E * C_alloc
    dt = torch.float32 if shape.x_dtype == F32 else torch.bfloat16
    _want(x, dt, shape.T * shape.H, "x")
    _want(inv, torch.int32, rows, "inv")
    _want(slot, torch.int32, shape.T, "slot")
    table, n = _ptr_table(peer_bufs)
    if window is not None:
        return _check("locmoe_dispatch_peer_window", _lib.locmoe_dispatch_peer_window(
            C.byref(shape), int(C_alloc), _ptr(x), _ptr(inv), _ptr(slot), table, n, int(src_lo), int(src_hi),
            1 if zero_pad else 0, int(window[0]), int(window[1]), _stream(stream)))
    return _check("locmoe_dispatch_peer", _lib.locmoe_dispatch_peer(C.byref(shape), int(C_alloc), _ptr(x), _ptr(inv), _ptr(slot),
                                                                    table, n, int(src_lo), int(src_hi), 1 if zero_pad else 0,
                                                                    _stream(stream)))


def locmoe_combine_peer(shape: Shape, C_alloc, peer_y, y_dtype, slot, gate_w, out, stream=None) -> int:
    dt = torch.float32 if shape.x_dtype == F32 else torch.bfloat16
    _want(slot, torch.int32, shape.T, "slot")
    _want(gate_w, torch.float32, shape.T, "gate_w")
    _want(out, dt, shape.T * shape.H, "out")
    table, n = _ptr_table(peer_y)
    return _check("locmoe_combine_peer", _lib.locmoe_combine_peer(C.byref(shape), int(C_alloc), table, n, int(y_dtype), _ptr(slot),
                                                                  _ptr(gate_w), _ptr(out), _stream(stream)))


def locmoe_topk_select(shape: Shape, probs, idx, gate_w, K, idx_k, w_k, stream=None) -> int:
    _want(probs, torch.float32, shape.T * shape.E, "probs")
    _want(idx, torch.int32, shape.T, "idx")
    _want(gate_w, torch.float32, shape.T, "gate_w")
    _want(idx_k, torch.int32, K * shape.T, "idx_k")
    _want(w_k, torch.float32, K * shape.T, "w_k")
    return _check("locmoe_topk_select", _lib.locmoe_topk_select(C.byref(shape), _ptr(probs), _ptr(idx), _ptr(gate_w), int(K),
                                                                _ptr(idx_k), _ptr(w_k), _stream(stream)))


def locmoe_topk_fold(shape: Shape, C_alloc, inv, stream=None) -> int:
    _want(inv, torch.int32, shape.D * shape.E * C_alloc, "inv")
    return _check("locmoe_topk_fold", _lib.locmoe_topk_fold(C.byref(shape), int(C_alloc), _ptr(inv), _stream(stream)))


def locmoe_combine_topk(shape: Shape, C_alloc, y, K, slot_k, w_k, out, stream=None) -> int:
    rows = shape.D * shape.E * C_alloc
    dt = torch.float32 if shape.x_dtype == F32 else torch.bfloat16
    _want(y, y.dtype, rows * shape.H, "y")
    _want(slot_k, torch.int32, K * shape.T, "slot_k")
    _want(w_k, torch.float32, K * shape.T, "w_k")
    _want(out, dt, shape.T * shape.H, "out")
    return _check("locmoe_combine_topk", _lib.locmoe_combine_topk(C.byref(shape), int(C_alloc), _ptr(y), dtype_code(y.dtype), int(K),
                                                                  _ptr(slot_k), _ptr(w_k), _ptr(out), _stream(stream)))


def locmoe_loc_loss(shape: Shape, counts, level, mu, smooth, dc_out, kl_out, group_tokens, loss_out, stream=None) -> int:
    G = shape.n_nodes if level else shape.D
    _want(counts, torch.int32, shape.D * shape.E, "counts")
    _want(dc_out, torch.float32, G * shape.E, "dc_out")
    _want(kl_out, torch.float64, G, "kl_out")
    _want(group_tokens, torch.int64, G, "group_tokens")
    _want(loss_out, torch.float64, 1, "loss_out")
    return _check("locmoe_loc_loss", _lib.locmoe_loc_loss(C.byref(shape), _ptr(counts), int(level), float(mu), float(smooth),
                                                          _ptr(dc_out), _ptr(kl_out), _ptr(group_tokens), _ptr(loss_out),
                                                          _stream(stream)))


def locmoe_cos_hist(shape: Shape, x, idx, expert, other, nbins, lo, hi, hist_routed, hist_other, n_routed, stream=None) -> int:
    dt = torch.float32 if shape.x_dtype == F32 else torch.bfloat16
    _want(x, dt, shape.T * shape.H, "x")
    _want(idx, torch.int32, shape.T, "idx")
    _want(hist_routed, torch.int32, nbins, "hist_routed")
    _want(hist_other, torch.int32, nbins, "hist_other")
    _want(n_routed, torch.int32, 1, "n_routed")
    return _check("locmoe_cos_hist", _lib.locmoe_cos_hist(C.byref(shape), _ptr(x), _ptr(idx), int(expert), int(other),
                                                          int(nbins), float(lo), float(hi), _ptr(hist_routed),
                                                          _ptr(hist_other), _ptr(n_routed), _stream(stream)))


def layer_buffers(st: "RouterState", h1=None, y=None) -> LayerBuffers:
    """Pointer block for locmoe_moe_layer from a RouterState (plus the FFN scratch and output)."""
    p = lambda t: None if t is None else t.data_ptr()
    return LayerBuffers(p(st.idx), p(st.gate_w), p(st.cos_sim), p(st.delta_e), p(st.theta_e), p(st.cap_dev), p(st.pos),
                        p(st.slot), p(st.drop), p(st.inv), p(st.counts), p(st.kept), p(st.send_counts), p(st.load),
                        p(st.locality), p(st.status), p(st.ws), st.ws.numel(), p(st.buf), p(h1), p(y))


def locmoe_moe_layer(shape: Shape, x, src_dev, eps, rule: CapacityRule, C_alloc, F, w_in, w_out, bufs: LayerBuffers,
                     out, stream=None) -> int:
    return _check("locmoe_moe_layer", _lib.locmoe_moe_layer(
        C.byref(shape), _ptr(x), _ptr(src_dev), _ptr(eps), C.byref(rule), int(C_alloc), int(F), _ptr(w_in), _ptr(w_out),
        C.byref(bufs), _ptr(out), _stream(stream)))


def conventional_capacity(T: int, D: int, E: int, capacity_factor: float) -> int:
    """Row stride to allocate the buffer with: the conventional term of the capacity rule for a batch of T tokens
    (``locmoe_conventional_capacity``; Sec. 3.2.3), evaluated by the library exactly as the device evaluates it."""
    shape = Shape(int(T), int(E), int(E), int(D), 1, F32, LAYOUT_SEND)      # only T, E and D enter the rule
    rule = CapacityRule(float(capacity_factor), float(capacity_factor), -1.0, BOUND_BETA, 0)
    out = C.c_int32(0)
    _check("locmoe_conventional_capacity", _lib.locmoe_conventional_capacity(C.byref(shape), C.byref(rule), C.byref(out)))
    return out.value


def batch_delta(delta_e) -> float:
    """Batch-wide cosine threshold from per-expert minima in HOST memory (``locmoe_batch_delta``): the minimum over
    the experts, clamped to [0, 1] as the device clamps it."""
    d = delta_e.detach().to("cpu", torch.float32).contiguous()
    out = C.c_double(0.0)
    _check("locmoe_batch_delta", _lib.locmoe_batch_delta(C.c_void_p(d.data_ptr()), int(d.numel()), C.byref(out)))
    return out.value


def dest_order(n_nodes: int, dev_per_node: int, a: int, b: int) -> int:
    """r(a, b): position of logical device b in device a's destination list (``locmoe_dest_order``)."""
    shape = Shape(1, 1, 1, int(n_nodes), int(dev_per_node), F32, LAYOUT_SEND)   # only the device map is read
    return _check("locmoe_dest_order", _lib.locmoe_dest_order(C.byref(shape), int(a), int(b)))


@dataclass
class RouterState:
    """Device buffers of one router instance (allocated once, reused every step)."""
    shape: Shape
    C_alloc: int
    rule: CapacityRule
    idx: torch.Tensor
    gate_w: torch.Tensor
    cos_sim: torch.Tensor
    delta_e: torch.Tensor
    theta_e: torch.Tensor
    cap_dev: torch.Tensor
    pos: torch.Tensor
    slot: torch.Tensor
    drop: torch.Tensor
    inv: torch.Tensor
    counts: torch.Tensor
    kept: torch.Tensor
    send_counts: torch.Tensor
    load: torch.Tensor
    locality: torch.Tensor
    status: torch.Tensor
    ws: torch.Tensor
    buf: torch.Tensor
    out: torch.Tensor

    @property
    def rows(self) -> int:
        return self.shape.D * self.shape.E * self.C_alloc


def make_router(shape: Shape, C_alloc: int, rule: CapacityRule, device="cuda", with_buffer: bool = True) -> RouterState:
    """Allocates every output and scratch tensor of the five calls with torch (memory plumbing only).
    ``with_buffer`` = False leaves out the dispatch buffer (a rank of the fused exchange writes into the peers'
    receive buffers instead)."""
    dev = torch.device(device)
    T, H, E, D = shape.T, shape.H, shape.E, shape.D
    rows = D * E * C_alloc
    xdt = torch.float32 if shape.x_dtype == F32 else torch.bfloat16
    i32 = dict(dtype=torch.int32, device=dev)
    f32 = dict(dtype=torch.float32, device=dev)
    ws_bytes = locmoe_workspace_bytes(shape, C_alloc)
    return RouterState(
        shape=shape, C_alloc=C_alloc, rule=rule,
        idx=torch.empty(T, **i32), gate_w=torch.empty(T, **f32), cos_sim=torch.empty(T, **f32),
        delta_e=torch.empty(E, **f32), theta_e=torch.empty(E, **f32),
        cap_dev=torch.zeros(CAPACITY_BYTES, dtype=torch.uint8, device=dev),
        pos=torch.empty(T, **i32), slot=torch.empty(T, **i32), drop=torch.empty(T, dtype=torch.uint8, device=dev),
        inv=torch.empty(rows, **i32), counts=torch.empty(D * E, **i32), kept=torch.empty(D * E, **i32),
        send_counts=torch.empty(D * D, **i32), load=torch.empty(E, **i32),
        locality=torch.empty(6, dtype=torch.int64, device=dev), status=torch.zeros(1, **i32),
        ws=torch.empty(ws_bytes, dtype=torch.uint8, device=dev),
        buf=torch.empty(rows if with_buffer else 0, H, dtype=xdt, device=dev), out=torch.empty(T, H, dtype=xdt, device=dev),
    )


def router_forward(st: RouterState, x, src_dev, y=None, eps=None, stream=None, out=None, fused=True):
    """gate -> capacity -> route -> dispatch -> combine on one stream.

    ``y`` are the expert outputs in slot layout; with ``y=None`` the experts are
    the identity and the dispatched buffer itself is combined.  ``fused`` = True runs the
    capacity and route stages as the single call ``locmoe_capacity_route``, "gate" runs
    gate, capacity and route as ``locmoe_gate_route``, False the three separate calls
    (same results).  Returns the combined output
    (``st.out`` unless ``out`` is given).
    """
    sh, Ca = st.shape, st.C_alloc
    out = st.out if out is None else out
    if fused == "gate":
        locmoe_gate_route(sh, x, eps, src_dev, st.rule, st, stream)
        locmoe_dispatch(sh, Ca, x, st.inv, st.buf, True, stream, slot=st.slot)
        locmoe_combine(sh, Ca, st.buf if y is None else y, st.slot, st.gate_w, out, False, stream)
        return out
    locmoe_gate(sh, x, eps, st.idx, st.gate_w, st.cos_sim, None, stream)
    if fused:
        locmoe_capacity_route(sh, st.idx, st.cos_sim, src_dev, st.rule, st.delta_e, st.theta_e, st.cap_dev, Ca, st.pos,
                              st.slot, st.drop, st.inv, st.counts, st.kept, st.send_counts, st.load, st.locality,
                              st.status, st.ws, stream, early_init=True)   # the kernel before it is the gate above
    else:
        locmoe_capacity(sh, st.idx, st.cos_sim, st.rule, st.delta_e, st.theta_e, st.cap_dev, st.ws, stream)
        locmoe_route(sh, st.idx, src_dev, st.cap_dev, Ca, st.pos, st.slot, st.drop, st.inv, st.counts, st.kept,
                     st.send_counts, st.load, st.locality, st.status, st.ws, stream)
    locmoe_dispatch(sh, Ca, x, st.inv, st.buf, True, stream, slot=st.slot)
    locmoe_combine(sh, Ca, st.buf if y is None else y, st.slot, st.gate_w, out, False, stream)
    return out


def make_topk_state(shape: Shape, K: int, C_alloc: int, device="cuda") -> dict:
    """Tensors of the top-k variant for T tokens and K choices (memory plumbing only)."""
    dev = torch.device(device)
    T, H, E, D = shape.T, shape.H, shape.E, shape.D
    i32 = dict(dtype=torch.int32, device=dev)
    f32 = dict(dtype=torch.float32, device=dev)
    xdt = torch.float32 if shape.x_dtype == F32 else torch.bfloat16
    shape_v = Shape(K * T, H, E, shape.n_nodes, shape.dev_per_node, shape.x_dtype, shape.layout)
    rows = D * E * C_alloc
    return dict(
        K=K, C_alloc=C_alloc, shape=shape, shape_v=shape_v,
        idx=torch.empty(T, **i32), gate_w=torch.empty(T, **f32), cos_sim=torch.empty(T, **f32), probs=torch.empty(T, E, **f32),
        delta_e=torch.empty(E, **f32), theta_e=torch.empty(E, **f32),
        cap_dev=torch.zeros(CAPACITY_BYTES, dtype=torch.uint8, device=dev),
        idx_k=torch.empty(K, T, **i32), w_k=torch.empty(K, T, **f32),
        pos=torch.empty(K, T, **i32), slot=torch.empty(K, T, **i32), drop=torch.empty(K, T, dtype=torch.uint8, device=dev),
        inv=torch.empty(rows, **i32), counts=torch.empty(D * E, **i32), kept=torch.empty(D * E, **i32),
        send_counts=torch.empty(D * D, **i32), load=torch.empty(E, **i32),
        locality=torch.empty(6, dtype=torch.int64, device=dev), status=torch.zeros(1, **i32),
        ws=torch.empty(max(locmoe_workspace_bytes(shape_v, C_alloc), locmoe_workspace_bytes(shape, C_alloc)),
                       dtype=torch.uint8, device=dev),
        buf=torch.empty(rows, H, dtype=xdt, device=dev), out=torch.empty(T, H, dtype=xdt, device=dev),
    )


def topk_forward(r: dict, x, src_k, rule: CapacityRule, y=None, stream=None, mark=None) -> dict:
    """The top-k variant on one stream: gate (with probabilities) -> capacity on the first choices, counting K * T
    assignments -> K best experts -> route of the K * T virtual tokens -> fold -> dispatch -> combine over the K
    choices.  ``src_k`` is the source-device array repeated K times; ``y`` are the expert outputs in slot layout
    (identity experts when None); ``mark`` is called between the stages (the bench records events there)."""
    shape, shape_v, K, C_alloc = r["shape"], r["shape_v"], r["K"], r["C_alloc"]
    mark = mark or (lambda: None)
    rule_k = CapacityRule(rule.min_mult, rule.capacity_factor, rule.delta_override, rule.bound_form, K * shape.T)
    mark()
    locmoe_gate(shape, x, None, r["idx"], r["gate_w"], r["cos_sim"], r["probs"], stream)
    mark()
    locmoe_capacity(shape, r["idx"], r["cos_sim"], rule_k, r["delta_e"], r["theta_e"], r["cap_dev"], r["ws"], stream)
    mark()
    locmoe_topk_select(shape, r["probs"], r["idx"], r["gate_w"], K, r["idx_k"], r["w_k"], stream)
    mark()
    locmoe_route(shape_v, r["idx_k"], src_k, r["cap_dev"], C_alloc, r["pos"], r["slot"], r["drop"], r["inv"],
                 r["counts"], r["kept"], r["send_counts"], r["load"], r["locality"], r["status"], r["ws"], stream)
    locmoe_topk_fold(shape, C_alloc, r["inv"], stream)
    mark()
    locmoe_dispatch(shape, C_alloc, x, r["inv"], r["buf"], True, stream)
    mark()
    locmoe_combine_topk(shape, C_alloc, r["buf"] if y is None else y, K, r["slot"], r["w_k"], r["out"], stream)
    mark()
    return r


def router_forward_topk(shape: Shape, x, src_dev, K: int, C_alloc: int, rule: CapacityRule, y=None, stream=None) -> dict:
    """Allocates the state and runs the top-k variant once (a convenience for tests and examples)."""
    r = make_topk_state(shape, K, C_alloc, x.device)
    r["src_k"] = src_dev.repeat(K).contiguous()
    return topk_forward(r, x, r["src_k"], rule, y=y, stream=stream)


class HostRouter:
    """The path for tokens that live in (pinned) host memory: copy in, five C-ABI calls, copy out.

    Successive ``forward`` calls are pipelined over three streams with double buffers: the host-to-device
    copy of step i+1 and the device-to-host copy of step i-1 run while step i computes, so a stream of
    batches is bound by one PCIe direction rather than by the sum of both copies and the kernels.
    Only memory and stream plumbing lives here; all arithmetic is in the library's kernels.
    """

    def __init__(self, shape: Shape, C_alloc: int, rule: CapacityRule, device="cuda"):
        dev = torch.device(device)
        self.st = make_router(shape, C_alloc, rule, dev)
        xdt = torch.float32 if shape.x_dtype == F32 else torch.bfloat16
        self.x = [torch.empty(shape.T, shape.H, dtype=xdt, device=dev) for _ in range(2)]
        self.src = [torch.empty(shape.T, dtype=torch.int32, device=dev) for _ in range(2)]
        self.out = [self.st.out, torch.empty_like(self.st.out)]
        self.s_in, self.s_comp, self.s_out = (torch.cuda.Stream(dev) for _ in range(3))
        self.ev_in = [torch.cuda.Event() for _ in range(2)]
        self.ev_comp = [torch.cuda.Event() for _ in range(2)]
        self.ev_out = [torch.cuda.Event() for _ in range(2)]
        self.i = 0

    def forward(self, x_host, src_host, out_host, y=None):
        """Queues one step; ``out_host`` is valid after ``synchronize()`` (or once a later step has reused its slot)."""
        k = self.i & 1
        with torch.cuda.stream(self.s_in):
            if self.i >= 2:
                self.s_in.wait_event(self.ev_comp[k])      # step i-2 has finished reading this input buffer
            self.x[k].copy_(x_host, non_blocking=True)
            self.src[k].copy_(src_host, non_blocking=True)
            self.ev_in[k].record(self.s_in)
        with torch.cuda.stream(self.s_comp):
            self.s_comp.wait_event(self.ev_in[k])
            if self.i >= 2:
                self.s_comp.wait_event(self.ev_out[k])     # step i-2's output has left this output buffer
            router_forward(self.st, self.x[k], self.src[k], y=y, stream=self.s_comp, out=self.out[k])
            self.ev_comp[k].record(self.s_comp)
        with torch.cuda.stream(self.s_out):
            self.s_out.wait_event(self.ev_comp[k])
            out_host.copy_(self.out[k], non_blocking=True)
            self.ev_out[k].record(self.s_out)
        self.i += 1

    def synchronize(self):
        for s in (self.s_in, self.s_comp, self.s_out):
            s.synchronize()
