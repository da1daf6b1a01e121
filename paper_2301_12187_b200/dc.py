"""ctypes binding of libdepthc (include/dc.h).  Argument marshalling only: every step of the
path runs in the library's CUDA kernels.  torch is used for device memory and streams.

The functions carry the names of the C entry points without the `dc_` prefix.  Importing this
module does not load the library; the first call does, and raises if it cannot.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence, Tuple

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libdepthc.so")

OK, ERR_INVALID_ARG, ERR_SHAPE, ERR_UNSUPPORTED, ERR_NOT_MERGEABLE, ERR_WORKSPACE, ERR_ALIGNMENT, \
    ERR_CUDA, ERR_TIMEOUT = range(9)
F32, BF16 = 0, 1
ACT_IDENTITY, ACT_RELU6 = 0, 1
ALGO_AUTO, ALGO_TCGEN05, ALGO_SIMT = 0, 1, 2
MERGE_AUTO, MERGE_STEPS = 0, 1

_FP = C.POINTER(C.c_float)


class Layer(C.Structure):
    _fields_ = [("c_in", C.c_int), ("c_out", C.c_int), ("groups", C.c_int),
                ("k", C.c_int), ("stride", C.c_int), ("pad", C.c_int),
                ("weight", C.c_void_p), ("bias", C.c_void_p),
                ("bn_gamma", C.c_void_p), ("bn_beta", C.c_void_p),
                ("bn_mean", C.c_void_p), ("bn_var", C.c_void_p), ("bn_eps", C.c_float)]


class Residual(C.Structure):
    _fields_ = [("first", C.c_int), ("last", C.c_int)]


class Geom(C.Structure):
    _fields_ = [("c_in", C.c_int), ("c_out", C.c_int), ("groups", C.c_int),
                ("k", C.c_int), ("stride", C.c_int), ("pad", C.c_int)]

    def as_tuple(self):
        return (self.c_in, self.c_out, self.groups, self.k, self.stride, self.pad)


class Block(C.Structure):
    _fields_ = [("c_in", C.c_int), ("c_hidden", C.c_int), ("c_out", C.c_int), ("has_expand", C.c_int),
                ("dw_k", C.c_int), ("dw_stride", C.c_int), ("dw_pad", C.c_int), ("has_residual", C.c_int),
                ("act_expand", C.c_int), ("act_dw", C.c_int),
                ("w_expand", C.c_void_p), ("b_expand", C.c_void_p), ("w_dw", C.c_void_p),
                ("b_dw", C.c_void_p), ("w_project", C.c_void_p), ("b_project", C.c_void_p)]


EXPORTS = {
    "dc_status_string": (C.c_char_p, [C.c_int]),
    "dc_fold_bn": (C.c_int, [C.POINTER(Layer), C.c_void_p, C.c_void_p, C.c_void_p]),
    "dc_merge_query": (C.c_int, [C.POINTER(Layer), C.c_int, C.POINTER(Residual), C.c_int,
                                 C.POINTER(Geom), C.POINTER(C.c_size_t)]),
    "dc_packed_bytes": (C.c_int, [C.POINTER(Geom), C.c_int, C.POINTER(C.c_size_t)]),
    "dc_merge_chain": (C.c_int, [C.POINTER(Layer), C.c_int, C.POINTER(Residual), C.c_int, C.c_void_p,
                                 C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_size_t, C.c_void_p]),
    "dc_merge_chain_algo": (C.c_int, [C.POINTER(Layer), C.c_int, C.POINTER(Residual), C.c_int, C.c_void_p,
                                      C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_size_t, C.c_void_p, C.c_int]),
    "dc_dp_optimal_latency": (C.c_int, [C.POINTER(C.c_longlong), C.c_int, C.POINTER(C.c_longlong), C.POINTER(C.c_int)]),
    "dc_dp_pattern": (C.c_int, [C.POINTER(C.c_int), C.c_int, C.c_int, C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_int)]),
    "dc_dp_select": (C.c_int, [C.POINTER(C.c_longlong), C.POINTER(C.c_double), C.c_int, C.c_longlong,
                               C.POINTER(C.c_int), C.POINTER(C.c_int), C.POINTER(C.c_int), C.POINTER(C.c_int),
                               C.POINTER(C.c_double), C.POINTER(C.c_int)]),
    "dc_dp_optimal_importance": (C.c_int, [C.POINTER(C.c_double), C.POINTER(C.c_ubyte), C.c_int, C.POINTER(C.c_double),
                                          C.POINTER(C.c_int)]),
    "dc_dp_importance_pattern": (C.c_int, [C.POINTER(C.c_int), C.c_int, C.c_int, C.c_int, C.c_int, C.c_int,
                                          C.POINTER(C.c_int), C.POINTER(C.c_int)]),
    "dc_dp_normalize_importance": (C.c_int, [C.POINTER(C.c_double), C.c_int, C.POINTER(C.c_double), C.c_int, C.c_double]),
    "dc_dp_select_ext": (C.c_int, [C.POINTER(C.c_longlong), C.POINTER(C.c_double), C.POINTER(C.c_ubyte), C.c_int,
                                  C.c_longlong, C.POINTER(C.c_int), C.POINTER(C.c_int), C.POINTER(C.c_int),
                                  C.POINTER(C.c_int), C.POINTER(C.c_int), C.POINTER(C.c_int), C.POINTER(C.c_int),
                                  C.POINTER(C.c_int), C.POINTER(C.c_double), C.POINTER(C.c_int)]),
    "dc_merge_chain_static": (C.c_int, [C.POINTER(Layer), C.c_int, C.POINTER(Residual), C.c_int, C.c_void_p,
                                        C.c_void_p, C.c_void_p, C.c_int, C.c_void_p]),
    "dc_merge_chain_static_capacity": (C.c_size_t, []),
    "dc_pack_weights": (C.c_int, [C.c_void_p, C.POINTER(Geom), C.c_int, C.c_void_p, C.c_void_p]),
    "dc_conv_workspace_bytes": (C.c_size_t, []),
    "dc_conv_kernel_name": (C.c_char_p, [C.c_int, C.c_int, C.c_int, C.POINTER(Geom), C.c_int]),
    "dc_conv_forward": (C.c_int, [C.c_void_p, C.c_int, C.c_int, C.c_int, C.POINTER(Geom), C.c_void_p,
                                  C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_int, C.c_void_p,
                                  C.c_size_t, C.c_void_p]),
    "dc_conv_forward_algo": (C.c_int, [C.c_void_p, C.c_int, C.c_int, C.c_int, C.POINTER(Geom), C.c_void_p,
                                       C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_int, C.c_void_p,
                                       C.c_size_t, C.c_void_p, C.c_int]),
    "dc_dwconv_forward": (C.c_int, [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int,
                                    C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.c_void_p]),
    "dc_dwconv_status": (C.c_int, [C.c_void_p]),
    "dc_block_workspace_bytes": (C.c_int, [C.c_int, C.c_int, C.c_int, C.POINTER(Block), C.c_int,
                                           C.POINTER(C.c_size_t)]),
    "dc_block_forward": (C.c_int, [C.c_void_p, C.c_int, C.c_int, C.c_int, C.POINTER(Block), C.c_void_p,
                                   C.c_int, C.c_void_p, C.c_size_t, C.c_void_p]),
    "dc_workspace_status": (C.c_int, [C.c_void_p, C.c_void_p]),
    "dc_workspace_status_where": (C.c_int, [C.c_void_p, C.c_void_p, C.POINTER(C.c_uint), C.POINTER(C.c_uint)]),
    "dc_selftest_bounded_wait": (C.c_int, [C.c_void_p, C.c_size_t, C.c_uint, C.c_void_p]),
    "dc_chain_host_param_layout": (C.c_int, [C.POINTER(Layer), C.c_int, C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]),
    "dc_chain_host_workspace_bytes": (C.c_int, [C.POINTER(Layer), C.c_int, C.POINTER(Residual), C.c_int,
                                                C.c_int, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_size_t)]),
    "dc_chain_forward_host": (C.c_int, [C.POINTER(Layer), C.c_int, C.POINTER(Residual), C.c_int, C.c_void_p,
                                        C.c_int, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_int, C.c_void_p,
                                        C.c_size_t, C.c_void_p]),
    "dc_chain_forward_host_async": (C.c_int, [C.POINTER(Layer), C.c_int, C.POINTER(Residual), C.c_int, C.c_void_p,
                                        C.c_int, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_int, C.c_void_p,
                                        C.c_size_t, C.c_void_p]),
}

_lib = None


class DcError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        try:
            msg = lib().dc_status_string(status).decode()
        except Exception:  # pragma: no cover
            msg = "?"
        super().__init__("%s: status %d (%s)" % (what, status, msg))


def lib():
    """Load libdepthc.so (building it with nvcc first if it is missing or stale).  Never falls
    back to anything else: without the library every call raises."""
    global _lib
    if _lib is None:
        from . import build as _build
        try:
            path = _build.build()
        except Exception as e:
            raise RuntimeError("libdepthc.so is missing and could not be built: %r" % (e,))
        L = C.CDLL(path)
        for name, (res, args) in EXPORTS.items():
            fn = getattr(L, name)
            fn.restype = res
            fn.argtypes = args
        _lib = L
    return _lib


def _check(st: int, what: str):
    if st != OK:
        raise DcError(st, what)


def _ptr(t) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream(stream=None) -> Optional[int]:
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    return stream.cuda_stream or None


def dtype_code(torch_dtype) -> int:
    import torch
    if torch_dtype == torch.float32:
        return F32
    if torch_dtype == torch.bfloat16:
        return BF16
    raise ValueError("dtype must be float32 or bfloat16")


def geom(c_in, c_out, groups, k, stride, pad) -> Geom:
    return Geom(c_in, c_out, groups, k, stride, pad)


class DeviceLayer:
    """One conv(+BN) with its parameters held as fp32 device tensors; `.c` is the dc_layer."""

    def __init__(self, spec, device="cuda"):
        import torch
        self.spec = spec
        self.tensors = {}

        def up(a):
            if a is None:
                return None
            return torch.from_numpy(a).to(device=device, dtype=torch.float32).contiguous()

        self.weight = up(spec.weight)
        self.bias = up(spec.bias)
        self.bn = None if spec.bn is None else tuple(up(t) for t in spec.bn)
        bn = self.bn or (None, None, None, None)
        self.c = Layer(spec.c_in, spec.c_out, spec.groups, spec.k, spec.stride, spec.pad,
                       _ptr(self.weight), _ptr(self.bias), _ptr(bn[0]), _ptr(bn[1]), _ptr(bn[2]),
                       _ptr(bn[3]), float(spec.eps))


def layer_array(layers: Sequence) -> "C.Array":
    """ctypes array of dc_layer from DeviceLayer objects or Layer structs."""
    arr = (Layer * len(layers))()
    for i, L in enumerate(layers):
        arr[i] = L.c if isinstance(L, DeviceLayer) else L
    return arr


def _res_array(residuals):
    residuals = list(residuals or [])
    arr = (Residual * max(1, len(residuals)))()
    for i, (f, l) in enumerate(residuals):
        arr[i] = Residual(f, l)
    return arr, len(residuals)


# --------------------------------------------------------------------------- entry points


def status_string(st: int) -> str:
    return lib().dc_status_string(st).decode()


def fold_bn(layer, w_out, b_out, stream=None):
    c = layer.c if isinstance(layer, DeviceLayer) else layer
    _check(lib().dc_fold_bn(C.byref(c), _ptr(w_out), _ptr(b_out), _stream(stream)), "dc_fold_bn")


def merge_query(layers, residuals=()) -> Tuple[Geom, int]:
    arr = layer_array(layers)
    res, n_res = _res_array(residuals)
    g = Geom()
    nbytes = C.c_size_t(0)
    _check(lib().dc_merge_query(arr, len(layers), res, n_res, C.byref(g), C.byref(nbytes)), "dc_merge_query")
    return g, int(nbytes.value)


def packed_bytes(g: Geom, dtype: int) -> int:
    nbytes = C.c_size_t(0)
    _check(lib().dc_packed_bytes(C.byref(g), dtype, C.byref(nbytes)), "dc_packed_bytes")
    return int(nbytes.value)


def merge_chain(layers, residuals, w_merged, b_merged, w_packed, packed_dtype, workspace, stream=None,
                algo=MERGE_AUTO):
    arr = layer_array(layers)
    res, n_res = _res_array(residuals)
    _check(lib().dc_merge_chain_algo(arr, len(layers), res, n_res, _ptr(w_merged), _ptr(b_merged),
                                     _ptr(w_packed), packed_dtype, _ptr(workspace),
                                     workspace.numel() * workspace.element_size(), _stream(stream), algo),
           "dc_merge_chain")


def merge_chain_static(layers, residuals, w_merged, b_merged, w_packed, packed_dtype, stream=None):
    """dc_merge_chain for callers that cannot allocate: the scratch is a fixed array inside the
    library (see include/dc.h for the limit and the sharing rules)."""
    arr = layer_array(layers)
    res, n_res = _res_array(residuals)
    _check(lib().dc_merge_chain_static(arr, len(layers), res, n_res, _ptr(w_merged), _ptr(b_merged),
                                       _ptr(w_packed), packed_dtype, _stream(stream)),
           "dc_merge_chain_static")


def merge_chain_static_capacity() -> int:
    return int(lib().dc_merge_chain_static_capacity())


DP_INF = 1 << 60


def _ll_table(T, L):
    flat = (C.c_longlong * ((L + 1) * (L + 1)))()
    for i in range(L + 1):
        for j in range(L + 1):
            flat[i * (L + 1) + j] = int(T[i][j]) if j > i else 0
    return flat


def dp_optimal_latency(T, L: int):
    """Algorithm 1 on host tables (lists or arrays indexed [i][j]): returns (T_opt, split) as lists
    of lists; split[k][l] is the last boundary of the optimal pattern of (k, l]."""
    W = L + 1
    t_opt = (C.c_longlong * (W * W))()
    split = (C.c_int * (W * W))()
    _check(lib().dc_dp_optimal_latency(_ll_table(T, L), L, t_opt, split), "dc_dp_optimal_latency")
    return ([[int(t_opt[i * W + j]) for j in range(W)] for i in range(W)],
            [[int(split[i * W + j]) for j in range(W)] for i in range(W)])


def dp_pattern(split, L: int, k: int, l: int):
    """S_opt[k][l] (increasing list) from the split table of dp_optimal_latency."""
    W = L + 1
    flat = (C.c_int * (W * W))(*[int(split[i][j]) for i in range(W) for j in range(W)])
    out = (C.c_int * max(L, 1))()
    n = C.c_int(0)
    _check(lib().dc_dp_pattern(flat, L, k, l, out, C.byref(n)), "dc_dp_pattern")
    return [int(out[i]) for i in range(n.value)]


def dp_select(T, I, L: int, T0: int):
    """Algorithm 2 on host tables: returns (A, S, objective, feasible)."""
    W = L + 1
    imp = (C.c_double * (W * W))()
    for i in range(W):
        for j in range(W):
            imp[i * W + j] = float(I[i][j]) if j > i else 0.0
    a = (C.c_int * max(L, 1))()
    s = (C.c_int * max(L, 1))()
    na, ns, ok = C.c_int(0), C.c_int(0), C.c_int(0)
    obj = C.c_double(0.0)
    _check(lib().dc_dp_select(_ll_table(T, L), imp, L, int(T0), a, C.byref(na), s, C.byref(ns), C.byref(obj),
                              C.byref(ok)), "dc_dp_select")
    return [int(a[i]) for i in range(na.value)], [int(s[i]) for i in range(ns.value)], obj.value, bool(ok.value)


def _imp4(I, L):
    W = L + 1
    flat = (C.c_double * (W * W * 4))()
    for i in range(W):
        for j in range(i + 1, W):
            for a in range(2):
                for b in range(2):
                    flat[((i * W + j) * 2 + a) * 2 + b] = float(I[i][j][a][b])
    return flat


def _flags(sigma_id, L):
    return (C.c_ubyte * (L + 1))(*[1 if x else 0 for x in sigma_id])


def dp_optimal_importance(I, sigma_id, L: int):
    """Algorithm 3 on host tables I[i][j][a][b]: returns (I_opt, split) as nested lists [k][l][a][b]."""
    W = L + 1
    out = (C.c_double * (W * W * 4))()
    split = (C.c_int * (W * W * 4))()
    _check(lib().dc_dp_optimal_importance(_imp4(I, L), _flags(sigma_id, L), L, out, split), "dc_dp_optimal_importance")
    nest = lambda f: [[[[f[((i * W + j) * 2 + a) * 2 + b] for b in range(2)] for a in range(2)] for j in range(W)]
                      for i in range(W)]
    return nest(out), nest(split)


def dp_importance_pattern(split, L: int, k: int, l: int, a: int, b: int):
    """B_opt[k][l][a][b] (increasing list) from the split table of dp_optimal_importance."""
    W = L + 1
    flat = (C.c_int * (W * W * 4))(*[int(split[i][j][x][y]) for i in range(W) for j in range(W) for x in range(2)
                                     for y in range(2)])
    out = (C.c_int * max(L, 1))()
    n = C.c_int(0)
    _check(lib().dc_dp_importance_pattern(flat, L, k, l, a, b, out, C.byref(n)), "dc_dp_importance_pattern")
    return [int(out[i]) for i in range(n.value)]


def dp_normalize_importance(I, L: int, deltas, alpha: float):
    """App. B.3 on a host table: returns the shifted copy as nested lists."""
    W = L + 1
    flat = _imp4(I, L)
    d = (C.c_double * len(deltas))(*[float(x) for x in deltas])
    _check(lib().dc_dp_normalize_importance(flat, L, d, len(deltas), float(alpha)), "dc_dp_normalize_importance")
    return [[[[flat[((i * W + j) * 2 + a) * 2 + b] for b in range(2)] for a in range(2)] for j in range(W)]
            for i in range(W)]


def dp_select_ext(T, I, sigma_id, L: int, T0: int):
    """Algorithm 4 on host tables: returns (A, S, B, d_first, d_last, objective, feasible)."""
    a = (C.c_int * max(L, 1))()
    s = (C.c_int * max(L, 1))()
    b = (C.c_int * max(L, 1))()
    na, ns, nb, d0, dl, ok = (C.c_int(0) for _ in range(6))
    obj = C.c_double(0.0)
    _check(lib().dc_dp_select_ext(_ll_table(T, L), _imp4(I, L), _flags(sigma_id, L), L, int(T0), a, C.byref(na), s,
                                  C.byref(ns), b, C.byref(nb), C.byref(d0), C.byref(dl), C.byref(obj), C.byref(ok)),
           "dc_dp_select_ext")
    return ([int(a[i]) for i in range(na.value)], [int(s[i]) for i in range(ns.value)],
            [int(b[i]) for i in range(nb.value)], d0.value, dl.value, obj.value, bool(ok.value))


def pack_weights(w, g: Geom, dtype: int, w_packed, stream=None):
    _check(lib().dc_pack_weights(_ptr(w), C.byref(g), dtype, _ptr(w_packed), _stream(stream)),
           "dc_pack_weights")


def conv_workspace_bytes() -> int:
    return int(lib().dc_conv_workspace_bytes())


def conv_kernel_name(n: int, h: int, w: int, g: Geom, dtype: int) -> Optional[str]:
    r = lib().dc_conv_kernel_name(n, h, w, C.byref(g), dtype)
    return r.decode() if r else None


def conv_forward(x, g: Geom, w_packed, bias, act, residual, y, workspace, stream=None, algo=ALGO_AUTO):
    n, h, w, _ = x.shape
    _check(lib().dc_conv_forward_algo(_ptr(x), n, h, w, C.byref(g), _ptr(w_packed), _ptr(bias), act,
                                      _ptr(residual), _ptr(y), dtype_code(x.dtype), _ptr(workspace),
                                      workspace.numel() * workspace.element_size(), _stream(stream), algo),
           "dc_conv_forward")


def dwconv_forward(x, k, stride, pad, w_packed, bias, act, y, stream=None):
    n, h, w, c = x.shape
    _check(lib().dc_dwconv_forward(_ptr(x), n, h, w, c, k, stride, pad, _ptr(w_packed), _ptr(bias), act,
                                   _ptr(y), dtype_code(x.dtype), _stream(stream)), "dc_dwconv_forward")


def dwconv_status(stream=None) -> int:
    return int(lib().dc_dwconv_status(_stream(stream)))


def block_workspace_bytes(n, h, w, blk: Block, dtype: int) -> int:
    nbytes = C.c_size_t(0)
    _check(lib().dc_block_workspace_bytes(n, h, w, C.byref(blk), dtype, C.byref(nbytes)),
           "dc_block_workspace_bytes")
    return int(nbytes.value)


def block_forward(x, blk: Block, y, workspace, stream=None):
    n, h, w, _ = x.shape
    _check(lib().dc_block_forward(_ptr(x), n, h, w, C.byref(blk), _ptr(y), dtype_code(x.dtype),
                                  _ptr(workspace), workspace.numel() * workspace.element_size(),
                                  _stream(stream)), "dc_block_forward")


def workspace_status(workspace, stream=None) -> int:
    return int(lib().dc_workspace_status(_ptr(workspace), _stream(stream)))


def workspace_status_where(workspace, stream=None) -> Tuple[int, int, int]:
    """(status, code of the wait that gave up, first detail word); clears the header like workspace_status."""
    where, detail = C.c_uint(0), C.c_uint(0)
    st = int(lib().dc_workspace_status_where(_ptr(workspace), _stream(stream), C.byref(where), C.byref(detail)))
    return st, int(where.value), int(detail.value)


def selftest_bounded_wait(workspace, limit_us: int, stream=None):
    _check(lib().dc_selftest_bounded_wait(_ptr(workspace), workspace.numel() * workspace.element_size(), int(limit_us),
                                          _stream(stream)), "dc_selftest_bounded_wait")


def host_layer_array(specs, pinned: bool = False) -> Tuple["C.Array", list]:
    """dc_layer array whose pointers are HOST pointers (float32), for chain_forward_host.  With
    pinned=True all arrays live in ONE page-locked block laid out as dc_chain_host_param_layout says,
    so their copy to the device is a single queued transfer instead of one staged copy per array."""
    import numpy as np
    keep = []
    arr = (Layer * len(specs))()
    for i, s in enumerate(specs):
        arr[i] = Layer(s.c_in, s.c_out, s.groups, s.k, s.stride, s.pad, None, None, None, None, None, None,
                       float(s.eps))
    block = None
    offs = (C.c_size_t * (6 * len(specs)))()
    if pinned:
        import torch
        total = C.c_size_t(0)
        _check(lib().dc_chain_host_param_layout(arr, len(specs), offs, C.byref(total)), "dc_chain_host_param_layout")
        block = torch.zeros(int(total.value), dtype=torch.uint8).pin_memory()
        keep.append(block)

    def hp(a, off):
        if a is None:
            return None
        a = np.ascontiguousarray(a, dtype=np.float32)
        if block is not None:
            import torch
            view = block[off:off + a.nbytes].view(torch.float32)
            view.copy_(torch.from_numpy(a.reshape(-1)))
            return block.data_ptr() + off
        keep.append(a)
        return a.ctypes.data

    for i, s in enumerate(specs):
        bn = s.bn or (None, None, None, None)
        arrays = (s.weight, s.bias, bn[0], bn[1], bn[2], bn[3])
        ptrs = [hp(a, int(offs[6 * i + j])) for j, a in enumerate(arrays)]
        arr[i].weight, arr[i].bias, arr[i].bn_gamma, arr[i].bn_beta, arr[i].bn_mean, arr[i].bn_var = ptrs
    return arr, keep


def chain_host_workspace_bytes(host_layers, n_layers, residuals, n, h, w, dtype: int) -> int:
    res, n_res = _res_array(residuals)
    nbytes = C.c_size_t(0)
    _check(lib().dc_chain_host_workspace_bytes(host_layers, n_layers, res, n_res, n, h, w, dtype,
                                               C.byref(nbytes)), "dc_chain_host_workspace_bytes")
    return int(nbytes.value)


def chain_forward_host(host_layers, n_layers, residuals, x_host, act, y_host, workspace, stream=None):
    """x_host / y_host: CPU torch tensors (pinned for asynchronous copies), NHWC."""
    res, n_res = _res_array(residuals)
    n, h, w, _ = x_host.shape
    _check(lib().dc_chain_forward_host(host_layers, n_layers, res, n_res, _ptr(x_host), n, h, w, act,
                                       _ptr(y_host), dtype_code(x_host.dtype), _ptr(workspace),
                                       workspace.numel() * workspace.element_size(), _stream(stream)),
           "dc_chain_forward_host")


def chain_forward_host_async(host_layers, n_layers, residuals, x_host, act, y_host, workspace, stream=None):
    """As chain_forward_host, but only queues the work on `stream`: keep every buffer alive and untouched
    until that stream has been synchronised."""
    res, n_res = _res_array(residuals)
    n, h, w, _ = x_host.shape
    _check(lib().dc_chain_forward_host_async(host_layers, n_layers, res, n_res, _ptr(x_host), n, h, w, act,
                                       _ptr(y_host), dtype_code(x_host.dtype), _ptr(workspace),
                                       workspace.numel() * workspace.element_size(), _stream(stream)),
           "dc_chain_forward_host_async")
