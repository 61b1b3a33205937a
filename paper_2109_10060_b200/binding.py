"""ctypes binding of libdsn: same names as the C ABI, argument marshalling only.

Tensors are torch CUDA tensors (PyTorch supplies device memory and streams, nothing else);
slice-width lists are Python ints.  Every compute step runs inside the library's kernels.
Loading fails loudly when the shared library has not been built.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(PKG_DIR, "libdsn.so")

OK = 0
ERR_INVALID_ARG, ERR_ALIGNMENT, ERR_WORKSPACE, ERR_UNSUPPORTED = -1, -2, -3, -4
ERR_BAD_INDEX, ERR_CUDA, ERR_TIMEOUT, ERR_NONFINITE = -5, -6, -7, -8
F32, BF16 = 0, 1
ACT_NONE, ACT_RELU, ACT_GELU = 0, 1, 2
INPUT_ORDER, GROUPED = 0, 1
TAIL_UNTOUCHED, TAIL_ZERO = 0, 1
LAYER_LINEAR, LAYER_CONV, LAYER_ATTENTION, LAYER_DEPTHWISE = 0, 1, 2, 3
MAX_SLICES, MAX_GROUPS, MAX_CHAIN = 64, 4096, 6

EXPORTS = [
    "dsn_create", "dsn_destroy", "dsn_strerror", "dsn_get_status", "dsn_set_wait_limit", "dsn_selftest_bounded_wait", "dsn_map_cache_stats", "dsn_get_stats", "dsn_widths_from_ratios",
    "dsn_executed_macs", "dsn_gate_workspace_bytes", "dsn_gate", "dsn_gate_static", "dsn_gate_attention", "dsn_scale_channels", "dsn_resbn_fold", "dsn_route", "dsn_permute_rows",
    "dsn_sliced_attention", "dsn_sliced_depthwise", "dsn_linear_workspace_bytes", "dsn_conv_workspace_bytes", "dsn_sliced_linear", "dsn_sliced_conv",
    "dsn_layer_workspace_bytes", "dsn_layer_forward",
]


class DsnError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: dsn status {code}")
        self.code = code


class Routing(C.Structure):
    _fields_ = [("B", C.c_int32), ("G", C.c_int32), ("counts", C.c_void_p), ("offsets", C.c_void_p),
                ("perm", C.c_void_p), ("inv_perm", C.c_void_p), ("group_slice", C.c_void_p)]


class GateDesc(C.Structure):
    _fields_ = [("dtype", C.c_int32), ("B", C.c_int32), ("R", C.c_int32), ("C_full", C.c_int32),
                ("c_valid", C.c_int32), ("C_mlp", C.c_int32), ("T", C.c_int32), ("ldx", C.c_int64),
                ("W1", C.c_void_p), ("b1", C.c_void_p), ("W2", C.c_void_p), ("b2", C.c_void_p)]


class LinearDesc(C.Structure):
    _fields_ = [("dtype", C.c_int32), ("R", C.c_int32), ("C_in", C.c_int32), ("C_out", C.c_int32),
                ("ldx", C.c_int64), ("ldw", C.c_int64), ("ldy", C.c_int64), ("T", C.c_int32),
                ("k_in", C.POINTER(C.c_int32)), ("k_out", C.POINTER(C.c_int32)), ("W", C.c_void_p),
                ("bias", C.c_void_p), ("bn_scale", C.c_void_p), ("bn_shift", C.c_void_p), ("residual", C.c_void_p),
                ("act", C.c_int32), ("in_order", C.c_int32), ("out_order", C.c_int32), ("tail", C.c_int32)]


class ConvDesc(C.Structure):
    _fields_ = [("dtype", C.c_int32), ("H", C.c_int32), ("W_", C.c_int32), ("K", C.c_int32), ("pad", C.c_int32),
                ("C_in", C.c_int32), ("C_out", C.c_int32), ("ldx", C.c_int64), ("ldy", C.c_int64),
                ("T", C.c_int32), ("k_in", C.POINTER(C.c_int32)), ("k_out", C.POINTER(C.c_int32)),
                ("W", C.c_void_p), ("bias", C.c_void_p), ("bn_scale", C.c_void_p), ("bn_shift", C.c_void_p),
                ("residual", C.c_void_p), ("act", C.c_int32), ("in_order", C.c_int32), ("out_order", C.c_int32),
                ("tail", C.c_int32)]


class AttentionDesc(C.Structure):
    _fields_ = [("dtype", C.c_int32), ("N", C.c_int32), ("H", C.c_int32), ("D_h", C.c_int32), ("ld_qkv", C.c_int64),
                ("ld_out", C.c_int64), ("T", C.c_int32), ("heads", C.POINTER(C.c_int32)), ("order", C.c_int32)]


class DepthwiseDesc(C.Structure):
    _fields_ = [("dtype", C.c_int32), ("H", C.c_int32), ("W_", C.c_int32), ("K", C.c_int32), ("stride", C.c_int32),
                ("C", C.c_int32), ("ldx", C.c_int64), ("ldy", C.c_int64), ("T", C.c_int32),
                ("c", C.POINTER(C.c_int32)), ("ksize", C.POINTER(C.c_int32)), ("W", C.c_void_p), ("bias", C.c_void_p),
                ("bn_scale", C.c_void_p), ("bn_shift", C.c_void_p), ("act", C.c_int32), ("in_order", C.c_int32),
                ("out_order", C.c_int32)]


class Stats(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in ("calls", "launches", "launches_gemm_pair", "launches_gemm_halo", "launches_gemm_chain",
                                          "launches_gemm_one_cta", "launches_linear_f32", "launches_attention",
                                          "launches_depthwise", "launches_dwpw", "launches_gate", "launches_route",
                                          "launches_copy", "map_hits", "map_misses", "launches_gemm_chain_tmem")]


class LayerDesc(C.Structure):
    _fields_ = [("gate", C.POINTER(GateDesc)), ("B", C.c_int32), ("T", C.c_int32), ("n_layers", C.c_int32),
                ("kind", C.c_int32 * MAX_CHAIN), ("layer", C.c_void_p * MAX_CHAIN)]


_lib = None


def load_library():
    """Loads libdsn.so (building it is `python -m paper_2109_10060_b200.build`)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2109_10060_b200.build`; "
                          "there is no fallback path")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
    lib.dsn_create.argtypes = [C.POINTER(vp), C.c_int]
    lib.dsn_destroy.argtypes = [vp]
    lib.dsn_strerror.argtypes = [C.c_int]
    lib.dsn_strerror.restype = C.c_char_p
    lib.dsn_get_status.argtypes = [vp, vp, C.POINTER(i32), C.POINTER(i32)]
    lib.dsn_set_wait_limit.argtypes = [vp, C.c_uint32, vp]
    lib.dsn_selftest_bounded_wait.argtypes = [vp, vp]
    lib.dsn_get_stats.argtypes = [vp, C.POINTER(Stats)]
    lib.dsn_map_cache_stats.argtypes = [vp, C.POINTER(C.c_uint64), C.POINTER(C.c_uint64)]
    lib.dsn_widths_from_ratios.argtypes = [i32, C.POINTER(C.c_double), i32, i32, C.POINTER(i32)]
    lib.dsn_executed_macs.argtypes = [C.POINTER(i32), i32, i32, C.POINTER(i32), C.POINTER(i32), i32]
    lib.dsn_executed_macs.restype = i64
    lib.dsn_gate_workspace_bytes.argtypes = [C.POINTER(GateDesc)]
    lib.dsn_gate_workspace_bytes.restype = sz
    lib.dsn_gate.argtypes = [vp, C.POINTER(GateDesc), vp, vp, vp, vp, sz, vp]
    lib.dsn_gate_static.argtypes = [vp, C.POINTER(GateDesc), vp, vp, vp, vp]
    lib.dsn_gate_attention.argtypes = [vp, C.POINTER(GateDesc), vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.dsn_scale_channels.argtypes = [vp, C.POINTER(Routing), i32, i32, i32, i32, i32, vp, i64, vp, vp, i64, vp]
    lib.dsn_resbn_fold.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, vp, vp]
    lib.dsn_route.argtypes = [vp, vp, i32, i32, C.POINTER(Routing), vp]
    lib.dsn_permute_rows.argtypes = [vp, C.POINTER(Routing), i32, i32, i32, C.POINTER(i32), vp, i64, vp, i64, i32, vp]
    lib.dsn_linear_workspace_bytes.argtypes = [C.POINTER(LinearDesc), i32]
    lib.dsn_linear_workspace_bytes.restype = sz
    lib.dsn_conv_workspace_bytes.argtypes = [C.POINTER(ConvDesc), i32]
    lib.dsn_conv_workspace_bytes.restype = sz
    lib.dsn_sliced_linear.argtypes = [vp, C.POINTER(LinearDesc), C.POINTER(Routing), vp, vp, vp, sz, vp]
    lib.dsn_sliced_conv.argtypes = [vp, C.POINTER(ConvDesc), C.POINTER(Routing), vp, vp, vp, sz, vp]
    lib.dsn_sliced_attention.argtypes = [vp, C.POINTER(AttentionDesc), C.POINTER(Routing), vp, vp, vp]
    lib.dsn_sliced_depthwise.argtypes = [vp, C.POINTER(DepthwiseDesc), C.POINTER(Routing), vp, vp, vp]
    lib.dsn_layer_workspace_bytes.argtypes = [C.POINTER(LayerDesc)]
    lib.dsn_layer_workspace_bytes.restype = sz
    lib.dsn_layer_forward.argtypes = [vp, C.POINTER(LayerDesc), vp, vp, vp, C.POINTER(Routing), vp, vp, sz, vp]
    for name in EXPORTS:
        fn = getattr(lib, name)
        if name not in ("dsn_strerror", "dsn_executed_macs") and not name.endswith("workspace_bytes"):
            fn.restype = C.c_int
    _lib = lib
    return lib


def _ptr(t) -> Optional[int]:
    return None if t is None else int(t.data_ptr())


def _i32_array(vals: Sequence[int]):
    return (C.c_int32 * len(vals))(*[int(v) for v in vals])


def _check(code: int, what: str):
    if code != OK:
        raise DsnError(code, what)


def _stream_handle(stream) -> Optional[int]:
    if stream is None:
        import torch
        return int(torch.cuda.current_stream().cuda_stream) or None
    return int(stream.cuda_stream) or None


def dsn_strerror(code: int) -> str:
    return load_library().dsn_strerror(code).decode()


def dsn_widths_from_ratios(C_full: int, ratios: Sequence[float], granule: int = 0):
    lib = load_library()
    T = len(ratios)
    out = (C.c_int32 * T)()
    _check(lib.dsn_widths_from_ratios(C_full, (C.c_double * T)(*ratios), T, granule, out), "dsn_widths_from_ratios")
    return list(out)


def dsn_executed_macs(counts: Sequence[int], R: int, k_in: Sequence[int], k_out: Sequence[int], K: int = 1) -> int:
    lib = load_library()
    return int(lib.dsn_executed_macs(_i32_array(counts), len(counts), R, _i32_array(k_in), _i32_array(k_out), K))


class Context:
    """Owns a dsn_ctx on one CUDA device."""

    def __init__(self, device: int = 0):
        self.lib = load_library()
        self.handle = C.c_void_p()
        _check(self.lib.dsn_create(C.byref(self.handle), device), "dsn_create")

    def close(self):
        if self.handle:
            self.lib.dsn_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_wait_limit(self, microseconds: int, stream=None):
        """Limit of the kernels' bounded waits (0 = the 2 s default)."""
        _check(self.lib.dsn_set_wait_limit(self.handle, int(microseconds), _stream_handle(stream)), "dsn_set_wait_limit")

    def selftest_bounded_wait(self, stream=None):
        """Launches the kernel that waits on a barrier nobody arrives at; it returns after the wait limit."""
        _check(self.lib.dsn_selftest_bounded_wait(self.handle, _stream_handle(stream)), "dsn_selftest_bounded_wait")

    def map_cache_stats(self):
        """(hits, misses) of the context's tensor-map cache."""
        h, m = C.c_uint64(), C.c_uint64()
        _check(self.lib.dsn_map_cache_stats(self.handle, C.byref(h), C.byref(m)), "dsn_map_cache_stats")
        return h.value, m.value

    def stats(self) -> dict:
        """Launch counters of this context (kernels of the library, by family)."""
        st = Stats()
        _check(self.lib.dsn_get_stats(self.handle, C.byref(st)), "dsn_get_stats")
        return {n: int(getattr(st, n)) for n, _ in Stats._fields_}

    def get_status(self, stream=None):
        code, detail = C.c_int32(), C.c_int32()
        _check(self.lib.dsn_get_status(self.handle, _stream_handle(stream), C.byref(code), C.byref(detail)),
               "dsn_get_status")
        return code.value, detail.value


def make_routing(B, G, counts, offsets, perm, inv_perm, group_slice=None) -> Routing:
    r = Routing(B, G, _ptr(counts), _ptr(offsets), _ptr(perm), _ptr(inv_perm), _ptr(group_slice))
    r._keep = (counts, offsets, perm, inv_perm, group_slice)
    return r


def make_gate_desc(dtype, B, R, C_full, C_mlp, T, W1, W2, b1=None, b2=None, c_valid=None, ldx=None) -> GateDesc:
    g = GateDesc(dtype, B, R, C_full, C_full if c_valid is None else c_valid, C_mlp, T,
                 C_full if ldx is None else ldx, _ptr(W1), _ptr(b1), _ptr(W2), _ptr(b2))
    g._keep = (W1, W2, b1, b2)
    return g


def make_linear_desc(dtype, R, C_in, C_out, k_in, k_out, W, bias=None, act=ACT_NONE, in_order=INPUT_ORDER,
                     out_order=INPUT_ORDER, tail=TAIL_UNTOUCHED, ldx=None, ldw=None, ldy=None, bn_scale=None,
                     bn_shift=None, residual=None) -> LinearDesc:
    ki, ko = _i32_array(k_in), _i32_array(k_out)
    d = LinearDesc(dtype, R, C_in, C_out, C_in if ldx is None else ldx, C_in if ldw is None else ldw,
                   C_out if ldy is None else ldy, len(k_in), ki, ko, _ptr(W), _ptr(bias), _ptr(bn_scale), _ptr(bn_shift),
                   _ptr(residual), act, in_order, out_order, tail)
    d._keep = (ki, ko, W, bias, bn_scale, bn_shift, residual)
    return d


def make_conv_desc(dtype, H, Wd, K, pad, C_in, C_out, k_in, k_out, W, bias=None, act=ACT_NONE,
                   in_order=INPUT_ORDER, out_order=INPUT_ORDER, tail=TAIL_UNTOUCHED, ldx=None, ldy=None, bn_scale=None,
                   bn_shift=None, residual=None) -> ConvDesc:
    ki, ko = _i32_array(k_in), _i32_array(k_out)
    d = ConvDesc(dtype, H, Wd, K, pad, C_in, C_out, C_in if ldx is None else ldx, C_out if ldy is None else ldy,
                 len(k_in), ki, ko, _ptr(W), _ptr(bias), _ptr(bn_scale), _ptr(bn_shift), _ptr(residual), act, in_order,
                 out_order, tail)
    d._keep = (ki, ko, W, bias, bn_scale, bn_shift, residual)
    return d


def make_layer_desc(B, T, layers, gate: Optional[GateDesc] = None) -> LayerDesc:
    L = LayerDesc()
    L.gate = C.pointer(gate) if gate is not None else None
    L.B, L.T, L.n_layers = B, T, len(layers)
    for j, d in enumerate(layers):
        L.kind[j] = (LAYER_CONV if isinstance(d, ConvDesc) else LAYER_ATTENTION if isinstance(d, AttentionDesc)
                     else LAYER_DEPTHWISE if isinstance(d, DepthwiseDesc) else LAYER_LINEAR)
        L.layer[j] = C.cast(C.pointer(d), C.c_void_p)
    L._keep = (gate, list(layers))
    return L


def dsn_gate_workspace_bytes(g: GateDesc) -> int:
    return int(load_library().dsn_gate_workspace_bytes(C.byref(g)))


def dsn_gate(ctx: Context, g: GateDesc, x, idx_out, logits_out=None, workspace=None, stream=None):
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(ctx.lib.dsn_gate(ctx.handle, C.byref(g), _ptr(x), _ptr(idx_out), _ptr(logits_out), _ptr(workspace),
                            ws_bytes, _stream_handle(stream)), "dsn_gate")


def dsn_gate_static(ctx: Context, g: GateDesc, x, idx_out, logits_out=None, stream=None):
    """dsn_gate without a workspace: for callers that may not allocate device memory (a serving loop
    that must stay out of the allocator, a plug-in that only receives its inputs and outputs).  The
    scratch is a fixed 4 MiB array inside the library, shared by all calls on a GPU, so calls must not
    overlap on the device, and problems beyond 1,048,576 scratch floats raise ERR_WORKSPACE."""
    _check(ctx.lib.dsn_gate_static(ctx.handle, C.byref(g), _ptr(x), _ptr(idx_out), _ptr(logits_out),
                                   _stream_handle(stream)), "dsn_gate_static")


def dsn_gate_attention(ctx: Context, g: GateDesc, W3, b3, x, idx_out, scale_out, logits_out=None, workspace=None,
                       stream=None):
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(ctx.lib.dsn_gate_attention(ctx.handle, C.byref(g), _ptr(W3), _ptr(b3), _ptr(x), _ptr(idx_out),
                                      _ptr(logits_out), _ptr(scale_out), _ptr(workspace), ws_bytes,
                                      _stream_handle(stream)), "dsn_gate_attention")


def dsn_scale_channels(ctx: Context, routing, to_grouped, dtype, B, R, c_valid, x, ldx, scale, y, ldy, stream=None):
    _check(ctx.lib.dsn_scale_channels(ctx.handle, C.byref(routing) if routing is not None else None,
                                      1 if to_grouped else 0, dtype, B, R, c_valid, _ptr(x), ldx, _ptr(scale), _ptr(y),
                                      ldy, _stream_handle(stream)), "dsn_scale_channels")


def dsn_resbn_fold(ctx: Context, T, Cn, gamma, beta, mu, sigma, scale_out, shift_out, stream=None):
    _check(ctx.lib.dsn_resbn_fold(ctx.handle, T, Cn, _ptr(gamma), _ptr(beta), _ptr(mu), _ptr(sigma), _ptr(scale_out),
                                  _ptr(shift_out), _stream_handle(stream)), "dsn_resbn_fold")


def dsn_route(ctx: Context, idx, B: int, T: int, routing: Routing, stream=None):
    _check(ctx.lib.dsn_route(ctx.handle, _ptr(idx), B, T, C.byref(routing), _stream_handle(stream)), "dsn_route")


def dsn_permute_rows(ctx: Context, routing: Routing, dtype, R, k, src, ld_src, dst, ld_dst, to_grouped, stream=None):
    _check(ctx.lib.dsn_permute_rows(ctx.handle, C.byref(routing), dtype, R, len(k), _i32_array(k), _ptr(src), ld_src,
                                    _ptr(dst), ld_dst, 1 if to_grouped else 0, _stream_handle(stream)),
           "dsn_permute_rows")


def dsn_sliced_linear(ctx: Context, d: LinearDesc, routing: Routing, x, y, workspace=None, stream=None):
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(ctx.lib.dsn_sliced_linear(ctx.handle, C.byref(d), C.byref(routing), _ptr(x), _ptr(y), _ptr(workspace),
                                     ws_bytes, _stream_handle(stream)), "dsn_sliced_linear")


def dsn_sliced_conv(ctx: Context, d: ConvDesc, routing: Routing, x, y, workspace=None, stream=None):
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(ctx.lib.dsn_sliced_conv(ctx.handle, C.byref(d), C.byref(routing), _ptr(x), _ptr(y), _ptr(workspace),
                                   ws_bytes, _stream_handle(stream)), "dsn_sliced_conv")


def make_attention_desc(N, H, D_h, heads, order=INPUT_ORDER, ld_qkv=None, ld_out=None) -> AttentionDesc:
    hs = _i32_array(heads)
    d = AttentionDesc(BF16, N, H, D_h, 3 * H * D_h if ld_qkv is None else ld_qkv, H * D_h if ld_out is None else ld_out,
                      len(heads), hs, order)
    d._keep = (hs,)
    return d


def dsn_sliced_attention(ctx: Context, d: AttentionDesc, routing: Routing, qkv, out, stream=None):
    _check(ctx.lib.dsn_sliced_attention(ctx.handle, C.byref(d), C.byref(routing), _ptr(qkv), _ptr(out),
                                        _stream_handle(stream)), "dsn_sliced_attention")


def make_depthwise_desc(H, Wd, K, stride, Cn, c, ksize, W, bias=None, act=ACT_NONE, in_order=INPUT_ORDER,
                        out_order=INPUT_ORDER, ldx=None, ldy=None, bn_scale=None, bn_shift=None) -> DepthwiseDesc:
    ca, ka = _i32_array(c), _i32_array(ksize)
    d = DepthwiseDesc(BF16, H, Wd, K, stride, Cn, Cn if ldx is None else ldx, Cn if ldy is None else ldy, len(c), ca, ka,
                      _ptr(W), _ptr(bias), _ptr(bn_scale), _ptr(bn_shift), act, in_order, out_order)
    d._keep = (ca, ka, W, bias, bn_scale, bn_shift)
    return d


def dsn_sliced_depthwise(ctx: Context, d: DepthwiseDesc, routing: Routing, x, y, stream=None):
    _check(ctx.lib.dsn_sliced_depthwise(ctx.handle, C.byref(d), C.byref(routing), _ptr(x), _ptr(y),
                                        _stream_handle(stream)), "dsn_sliced_depthwise")


def dsn_layer_workspace_bytes(L: LayerDesc) -> int:
    return int(load_library().dsn_layer_workspace_bytes(C.byref(L)))


def dsn_layer_forward(ctx: Context, L: LayerDesc, x, idx_in, y, workspace, r_out: Optional[Routing] = None,
                      idx_out=None, stream=None):
    ws_bytes = workspace.numel() * workspace.element_size()
    _check(ctx.lib.dsn_layer_forward(ctx.handle, C.byref(L), _ptr(x), _ptr(idx_in), _ptr(y),
                                     C.byref(r_out) if r_out is not None else None, _ptr(idx_out), _ptr(workspace),
                                     ws_bytes, _stream_handle(stream)), "dsn_layer_forward")
