"""Thin ctypes binding of ``libpipe.so`` (the C ABI of ``include/pipe.h``).

Argument marshalling only: every step of the path runs in the library's CUDA kernels.
PyTorch supplies device memory and streams; tensors are passed as raw device pointers.
There is no fallback: if the library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

from . import build as _build

MAX_ORDERS = 16
BLOCK_ROWS = 256
BLOCK_CHANNELS = 512
EVEN_BLOCKS = 8   # PIPE_EVEN_BLOCKS
BLOCK_RECORD_BYTES = 32 * 4 + 8 * (BLOCK_CHANNELS // 8) * 2 + BLOCK_ROWS * 4
BLOB_ALIGN = 1024

STATUS_NAMES = ["PIPE_OK", "PIPE_ERR_INVALID_ARG", "PIPE_ERR_SHAPE", "PIPE_ERR_ALIGNMENT", "PIPE_ERR_UNSUPPORTED",
                "PIPE_ERR_WORKSPACE", "PIPE_ERR_NONFINITE", "PIPE_ERR_ACC_OVERFLOW", "PIPE_ERR_TIMEOUT",
                "PIPE_ERR_CUDA"]
(PIPE_OK, PIPE_ERR_INVALID_ARG, PIPE_ERR_SHAPE, PIPE_ERR_ALIGNMENT, PIPE_ERR_UNSUPPORTED, PIPE_ERR_WORKSPACE,
 PIPE_ERR_NONFINITE, PIPE_ERR_ACC_OVERFLOW, PIPE_ERR_TIMEOUT, PIPE_ERR_CUDA) = range(10)

KERNEL_AUTO, KERNEL_REFERENCE, KERNEL_TCGEN05, KERNEL_STREAM, KERNEL_TCGEN05_PAIR, KERNEL_DECODE_TC = 0, 1, 2, 3, 4, 5

STATIC_SCRATCH_BYTES = 4 << 20

EXPORTS = ["pipe_keep_groups_from_gamma", "pipe_default_branches", "pipe_layout", "pipe_expand_weights",
           "pipe_bit_ops_original", "pipe_bit_ops_expanded", "pipe_max_orders_within_original", "pipe_gamma_from_budget",
           "pipe_bound_network", "pipe_bound_step_dense", "pipe_bound_step_rows", "pipe_spectral_norm", "pipe_choose_expansion",
           "pipe_expand_weights_static",
           "pipe_quantize_act", "pipe_quantize_act_ex", "pipe_ensemble_forward_zp", "pipe_expanded_linear", "pipe_expanded_conv2d", "pipe_ensemble_forward",
           "pipe_ensemble_forward_q8", "pipe_expanded_conv2d_q8", "pipe_ensemble_conv2d", "pipe_ensemble_conv2d_q8",
           "pipe_lower_conv_input",
           "pipe_launch_count", "pipe_poll_status", "pipe_status_string",
           # include/pipe_diag.h: tests and measurements only
           "pipe_diag_select_kernel", "pipe_diag_mma_i8_rate", "pipe_diag_bounded_wait"]


class LayerDesc(C.Structure):
    _fields_ = [("out_features", C.c_int32), ("in_features", C.c_int32), ("weight_bits", C.c_int32),
                ("num_orders", C.c_int32), ("group_size", C.c_int32), ("keep_groups", C.c_int32),
                ("num_branches", C.c_int32), ("branch_orders", C.c_int32 * MAX_ORDERS),
                ("score_mode", C.c_int32), ("keep_elems", C.c_int32), ("int8_copy", C.c_int32)]


class ConvGeom(C.Structure):
    _fields_ = [("batch", C.c_int32), ("height", C.c_int32), ("width", C.c_int32), ("channels", C.c_int32),
                ("kernel_h", C.c_int32), ("kernel_w", C.c_int32), ("pad_h", C.c_int32), ("pad_w", C.c_int32),
                ("stride_h", C.c_int32), ("stride_w", C.c_int32)]


class LayerLayout(C.Structure):
    _fields_ = [("num_groups", C.c_int32), ("total_rows", C.c_int32), ("canon_row_bytes", C.c_int32),
                ("kernel_row_bytes", C.c_int32), ("rows", C.c_int32 * MAX_ORDERS),
                ("kept_groups", C.c_int32 * MAX_ORDERS), ("branch_orders", C.c_int32 * MAX_ORDERS),
                ("codes_off", C.c_uint64 * MAX_ORDERS), ("kcodes_off", C.c_uint64 * MAX_ORDERS),
                ("wcodes_off", C.c_uint64 * MAX_ORDERS),
                ("scales_off", C.c_uint64 * MAX_ORDERS), ("kept_off", C.c_uint64 * MAX_ORDERS),
                ("cum_off", C.c_uint64 * MAX_ORDERS), ("blk_off", C.c_uint64 * (MAX_ORDERS + 1)),
                ("blk_cap", C.c_int32 * (MAX_ORDERS + 1)), ("rec_off", C.c_uint64 * (MAX_ORDERS + 1)),
                ("rec_cap", C.c_int32 * (MAX_ORDERS + 1)), ("decode_split", C.c_int32),
                ("dec_off", C.c_uint64 * (MAX_ORDERS + 1)), ("dec_limit", C.c_int32 * (MAX_ORDERS + 1)),
                ("decode_split_all", C.c_int32),
                ("blob_bytes", C.c_uint64), ("expand_ws_bytes", C.c_uint64),
                ("quantize_ws_bytes", C.c_uint64)]


class PipeError(RuntimeError):
    def __init__(self, status: int, where: str):
        name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        super().__init__(f"{where}: {name}")
        self.status = status


_lib = None


def library_path() -> str:
    return _build.LIB


def lib() -> C.CDLL:
    """Load libpipe.so (must have been built: ``python -m paper_2311_15806_b200.build``)."""
    global _lib
    if _lib is None:
        path = library_path()
        if not os.path.exists(path):
            raise RuntimeError(f"{path} not found: build the CUDA library first (python -m paper_2311_15806_b200.build)")
        L = C.CDLL(path)
        i32, i64, p, sz = C.c_int32, C.c_int64, C.c_void_p, C.c_size_t
        L.pipe_keep_groups_from_gamma.argtypes = [i32, C.c_double]
        L.pipe_keep_groups_from_gamma.restype = i32
        L.pipe_default_branches.argtypes = [i32, i32, p]
        L.pipe_layout.argtypes = [C.POINTER(LayerDesc), C.POINTER(LayerLayout)]
        L.pipe_expand_weights.argtypes = [C.POINTER(LayerDesc), p, i64, p, sz, p, sz, p]
        L.pipe_expand_weights_static.argtypes = [C.POINTER(LayerDesc), p, i64, p, sz, p]
        L.pipe_quantize_act.argtypes = [p, i64, i32, i64, p, p, i64, p, p, sz, p]
        L.pipe_quantize_act_ex.argtypes = [p, i64, i32, i64, i32, i32, p, p, p, i64, p, p, p, sz, p]
        L.pipe_ensemble_forward_zp.argtypes = [C.POINTER(LayerDesc), p, p, i64, i64, p, p, p, p, i64, i32, p, p]
        L.pipe_expanded_linear.argtypes = [C.POINTER(LayerDesc), p, p, i64, i64, p, p, p, i64, p, p]
        L.pipe_expanded_conv2d.argtypes = [C.POINTER(LayerDesc), C.POINTER(ConvGeom), p, p, p, p, p, i64, p, p]
        L.pipe_ensemble_forward.argtypes = [C.POINTER(LayerDesc), p, p, i64, i64, p, p, p, i64, i32, p, p]
        L.pipe_ensemble_forward_q8.argtypes = [C.POINTER(LayerDesc), p, p, i64, i64, p, p, i32, p, p, i64, p, p]
        L.pipe_expanded_conv2d_q8.argtypes = [C.POINTER(LayerDesc), C.POINTER(ConvGeom), p, p, p, p, i32, p, p, i64, p, p]
        L.pipe_ensemble_conv2d.argtypes = [C.POINTER(LayerDesc), C.POINTER(ConvGeom), p, p, p, p, p, i64, i32, p, p]
        L.pipe_ensemble_conv2d_q8.argtypes = [C.POINTER(LayerDesc), C.POINTER(ConvGeom), p, p, p, p, i32, p, p, i64, p, p]
        L.pipe_lower_conv_input.argtypes = [C.POINTER(ConvGeom), p, p, i64, p]
        L.pipe_diag_select_kernel.argtypes = [i32]
        L.pipe_diag_mma_i8_rate.argtypes = [i32, i64, i32, C.POINTER(C.c_double), p]
        L.pipe_diag_bounded_wait.argtypes = [i64, p]
        L.pipe_launch_count.restype = C.c_uint64
        L.pipe_poll_status.argtypes = [p, C.POINTER(i32)]
        L.pipe_status_string.argtypes = [C.c_int]
        L.pipe_status_string.restype = C.c_char_p
        _lib = L
    return _lib


def _check(status: int, where: str) -> None:
    if status != PIPE_OK:
        raise PipeError(status, where)


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def _dp(t) -> int | None:
    return None if t is None else int(t.data_ptr())


class OpShape(C.Structure):
    _fields_ = [("kernel_size", C.c_int32), ("feature_size", C.c_int32), ("in_channels", C.c_int32),
                ("out_channels", C.c_int32), ("stride", C.c_int32)]


def _op_shape(d: int, D: int, n_i: int, n_o: int, s: int) -> OpShape:
    return OpShape(int(d), int(D), int(n_i), int(n_o), int(s))


def pipe_bit_ops_original(d: int, D: int, n_i: int, n_o: int, s: int) -> float:
    L = lib()
    L.pipe_bit_ops_original.restype = C.c_double
    return float(L.pipe_bit_ops_original(C.byref(_op_shape(d, D, n_i, n_o, s))))


def pipe_bit_ops_expanded(d: int, D: int, n_i: int, n_o: int, s: int, bits: int, orders: float) -> float:
    L = lib()
    L.pipe_bit_ops_expanded.restype = C.c_double
    L.pipe_bit_ops_expanded.argtypes = [C.c_void_p, C.c_int32, C.c_double]
    return float(L.pipe_bit_ops_expanded(C.byref(_op_shape(d, D, n_i, n_o, s)), int(bits), float(orders)))


def pipe_max_orders_within_original(d: int, D: int, n_i: int, n_o: int, s: int, bits: int) -> int:
    L = lib()
    L.pipe_max_orders_within_original.restype = C.c_int32
    return int(L.pipe_max_orders_within_original(C.byref(_op_shape(d, D, n_i, n_o, s)), int(bits)))


def pipe_gamma_from_budget(beta: float, K: int) -> float:
    L = lib()
    L.pipe_gamma_from_budget.argtypes = [C.c_double, C.c_int32, C.c_void_p]
    out = C.c_double(0.0)
    _check(L.pipe_gamma_from_budget(float(beta), int(K), C.byref(out)), "pipe_gamma_from_budget")
    return float(out.value)


def pipe_bound_network(s, u) -> float:
    """U of Appendix C for spectral norms s and steps u (sequences of equal length)."""
    L = lib()
    L.pipe_bound_network.restype = C.c_double
    L.pipe_bound_network.argtypes = [C.c_void_p, C.c_void_p, C.c_int32]
    n = len(s)
    sa, ua = (C.c_double * n)(*[float(v) for v in s]), (C.c_double * n)(*[float(v) for v in u])
    return float(L.pipe_bound_network(sa, ua, n))


def pipe_bound_step_dense(bits: int, K: int, first_scale_max: float) -> float:
    L = lib()
    L.pipe_bound_step_dense.restype = C.c_double
    L.pipe_bound_step_dense.argtypes = [C.c_int32, C.c_int32, C.c_double]
    return float(L.pipe_bound_step_dense(int(bits), int(K), float(first_scale_max)))


def pipe_bound_step_rows(last_scale) -> float:
    """last_scale: host float32 array [O] (see last_kept_scales)."""
    import numpy as np
    L = lib()
    L.pipe_bound_step_rows.restype = C.c_double
    L.pipe_bound_step_rows.argtypes = [C.c_void_p, C.c_int32]
    a = np.ascontiguousarray(last_scale, dtype=np.float32)
    return float(L.pipe_bound_step_rows(a.ctypes.data_as(C.c_void_p), a.shape[0]))


def pipe_spectral_norm(W, max_iters: int = 200, tol: float = 1e-9) -> float:
    """W: host float32 array [O, I]."""
    import numpy as np
    L = lib()
    L.pipe_spectral_norm.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int64, C.c_int32, C.c_double, C.c_void_p]
    a = np.ascontiguousarray(W, dtype=np.float32)
    out = C.c_double(0.0)
    _check(L.pipe_spectral_norm(a.ctypes.data_as(C.c_void_p), a.shape[0], a.shape[1], a.shape[1], int(max_iters), float(tol),
                                C.byref(out)), "pipe_spectral_norm")
    return float(out.value)


def pipe_choose_expansion(d: int, D: int, n_i: int, n_o: int, s: int, bits: int, bit_ops_budget: float, max_orders: int,
                          min_gamma: float, num_branches: int):
    """Returns (K, gamma, [K_m])."""
    L = lib()
    L.pipe_choose_expansion.argtypes = [C.c_void_p, C.c_int32, C.c_double, C.c_int32, C.c_double, C.c_int32, C.c_void_p,
                                        C.c_void_p, C.c_void_p, C.c_void_p]
    K, M, g = C.c_int32(0), C.c_int32(0), C.c_double(0.0)
    bo = (C.c_int32 * MAX_ORDERS)()
    _check(L.pipe_choose_expansion(C.byref(_op_shape(d, D, n_i, n_o, s)), int(bits), float(bit_ops_budget), int(max_orders),
                                   float(min_gamma), int(num_branches), C.byref(K), C.byref(g), C.byref(M), bo),
           "pipe_choose_expansion")
    return int(K.value), float(g.value), [int(bo[m]) for m in range(M.value)]


def pipe_keep_groups_from_gamma(num_groups: int, gamma: float) -> int:
    return int(lib().pipe_keep_groups_from_gamma(num_groups, float(gamma)))


def pipe_default_branches(K: int, M: int) -> list[int]:
    out = (C.c_int32 * MAX_ORDERS)()
    _check(lib().pipe_default_branches(K, M, out), "pipe_default_branches")
    return [int(out[m]) for m in range(M)]


SCORE_MAXABS, SCORE_L2 = 0, 1
ACT_IDENTITY, ACT_RELU, ACT_SILU, ACT_GELU, ACT_SIGMOID = 0, 1, 2, 3, 4


def make_desc(O: int, I: int, bits: int, K: int, g: int, keep_groups: int, M: int = 1,
              branch_orders=None, score_mode: int = 0, keep_elems: int = 0, int8_copy: bool = False) -> LayerDesc:
    d = LayerDesc()
    d.out_features, d.in_features, d.weight_bits, d.num_orders = O, I, bits, K
    d.group_size, d.keep_groups, d.num_branches = g, keep_groups, M
    d.score_mode, d.keep_elems = score_mode, keep_elems
    d.int8_copy = 1 if int8_copy else 0
    if branch_orders is not None:
        for m, v in enumerate(branch_orders):
            d.branch_orders[m] = int(v)
    return d


def pipe_layout(desc: LayerDesc) -> LayerLayout:
    out = LayerLayout()
    _check(lib().pipe_layout(C.byref(desc), C.byref(out)), "pipe_layout")
    return out


def pipe_expand_weights(desc: LayerDesc, W: torch.Tensor, blob: torch.Tensor, ws: torch.Tensor, stream=None) -> None:
    """W: cuda float32 [O, I] (last dim contiguous); blob / ws: cuda uint8 buffers sized by pipe_layout."""
    assert W.is_cuda and W.dtype == torch.float32 and W.stride(1) == 1
    _check(lib().pipe_expand_weights(C.byref(desc), _dp(W), W.stride(0), _dp(blob), blob.numel(), _dp(ws), ws.numel(),
                                     _stream_ptr(stream)), "pipe_expand_weights")


def pipe_expand_weights_static(desc: LayerDesc, W: torch.Tensor, blob: torch.Tensor, stream=None) -> None:
    """pipe_expand_weights without a workspace argument: the library's fixed internal array
    (STATIC_SCRATCH_BYTES) is used instead, so the call allocates nothing.  Raises PipeError
    (PIPE_ERR_WORKSPACE) when the layer is too large for that array."""
    assert W.is_cuda and W.dtype == torch.float32 and W.stride(1) == 1
    _check(lib().pipe_expand_weights_static(C.byref(desc), _dp(W), W.stride(0), _dp(blob), blob.numel(),
                                            _stream_ptr(stream)), "pipe_expand_weights_static")


def pipe_quantize_act(x: torch.Tensor, xq: torch.Tensor, sx: torch.Tensor, ws: torch.Tensor,
                      static_scale: torch.Tensor | None = None, stream=None) -> None:
    """x: cuda float32 [T, I]; xq: cuda int8 [T, I]; sx: cuda float32 [1]; ws: cuda uint8 >= 256 bytes."""
    assert x.is_cuda and x.dtype == torch.float32 and xq.dtype == torch.int8
    T, I = x.shape
    ldx = x.stride(0) if T > 1 else max(I, x.stride(0))
    ldxq = xq.stride(0) if T > 1 else max(I, xq.stride(0))
    _check(lib().pipe_quantize_act(_dp(x), T, I, ldx, _dp(static_scale), _dp(xq), ldxq, _dp(sx), _dp(ws), ws.numel(),
                                   _stream_ptr(stream)), "pipe_quantize_act")


def pipe_quantize_act_ex(x: torch.Tensor, xq: torch.Tensor, sx: torch.Tensor, zp: torch.Tensor, ws: torch.Tensor, act_bits: int = 8,
                         asymmetric: bool = False, static_scale: torch.Tensor | None = None,
                         static_range: torch.Tensor | None = None, stream=None) -> None:
    """x: cuda float32 [T, I]; xq: cuda int8 [T, I]; sx: cuda float32 [1]; zp: cuda int32 [1]; ws: cuda uint8 >= 256 bytes."""
    assert x.is_cuda and x.dtype == torch.float32 and xq.dtype == torch.int8 and zp.dtype == torch.int32
    T, I = x.shape
    ldx = x.stride(0) if T > 1 else max(I, x.stride(0))
    ldxq = xq.stride(0) if T > 1 else max(I, xq.stride(0))
    _check(lib().pipe_quantize_act_ex(_dp(x), T, I, ldx, int(act_bits), 1 if asymmetric else 0, _dp(static_scale), _dp(static_range),
                                      _dp(xq), ldxq, _dp(sx), _dp(zp), _dp(ws), ws.numel(), _stream_ptr(stream)), "pipe_quantize_act_ex")


def pipe_ensemble_forward_zp(desc: LayerDesc, blob: torch.Tensor, xq_m, sx_m, zp_m, y_m, bias: torch.Tensor | None = None,
                             sum_branches: bool = False, partials: torch.Tensor | None = None, stream=None) -> None:
    """pipe_ensemble_forward on asymmetric codes; zp_m: sequence of M cuda int32 one-element tensors (or None entries)."""
    M = desc.num_branches
    assert len(xq_m) == M and len(sx_m) == M and len(zp_m) == M and len(y_m) >= (1 if sum_branches else M)
    T = xq_m[0].shape[0]
    ldxq = xq_m[0].stride(0) if T > 1 else max(xq_m[0].shape[1], xq_m[0].stride(0))
    ldy = y_m[0].stride(0) if T > 1 else max(y_m[0].shape[1], y_m[0].stride(0))
    PA = C.c_void_p * M
    xp = PA(*[_dp(t) for t in xq_m])
    sp = PA(*[_dp(t) for t in sx_m])
    zp = PA(*[_dp(t) for t in zp_m])
    yp = PA(*[(_dp(y_m[m]) if m < len(y_m) else None) for m in range(M)])
    _check(lib().pipe_ensemble_forward_zp(C.byref(desc), _dp(blob), xp, T, ldxq, sp, zp, _dp(bias), yp, ldy,
                                          1 if sum_branches else 0, _dp(partials), _stream_ptr(stream)),
           "pipe_ensemble_forward_zp")


def pipe_expanded_linear(desc: LayerDesc, blob: torch.Tensor, xq: torch.Tensor, sx: torch.Tensor, y: torch.Tensor,
                         bias: torch.Tensor | None = None, partials: torch.Tensor | None = None, stream=None) -> None:
    T = xq.shape[0]
    ldxq = xq.stride(0) if T > 1 else max(xq.shape[1], xq.stride(0))
    ldy = y.stride(0) if T > 1 else max(y.shape[1], y.stride(0))
    _check(lib().pipe_expanded_linear(C.byref(desc), _dp(blob), _dp(xq), T, ldxq, _dp(sx), _dp(bias), _dp(y), ldy,
                                      _dp(partials), _stream_ptr(stream)), "pipe_expanded_linear")


def pipe_expanded_conv2d(desc: LayerDesc, geom: ConvGeom, blob: torch.Tensor, xq_nhwc: torch.Tensor, sx: torch.Tensor,
                         y: torch.Tensor, bias: torch.Tensor | None = None, partials: torch.Tensor | None = None,
                         stream=None) -> None:
    """xq_nhwc: cuda int8 [N, H, W, C] contiguous; y: cuda float32 [N*Ho*Wo, O]."""
    assert xq_nhwc.is_contiguous() and xq_nhwc.dtype == torch.int8
    _check(lib().pipe_expanded_conv2d(C.byref(desc), C.byref(geom), _dp(blob), _dp(xq_nhwc), _dp(sx), _dp(bias), _dp(y),
                                      y.stride(0), _dp(partials), _stream_ptr(stream)), "pipe_expanded_conv2d")


def pipe_expanded_conv2d_q8(desc: LayerDesc, geom: ConvGeom, blob: torch.Tensor, xq_nhwc: torch.Tensor, sx: torch.Tensor,
                            out_scale: torch.Tensor, yq: torch.Tensor, bias: torch.Tensor | None = None, relu: bool = True,
                            partials: torch.Tensor | None = None, stream=None) -> None:
    """xq_nhwc: cuda int8 [N, H, W, C] contiguous; yq: cuda int8 [N*Ho*Wo, O]; out_scale: cuda float32, one element."""
    assert xq_nhwc.is_contiguous() and xq_nhwc.dtype == torch.int8 and yq.dtype == torch.int8
    _check(lib().pipe_expanded_conv2d_q8(C.byref(desc), C.byref(geom), _dp(blob), _dp(xq_nhwc), _dp(sx), _dp(bias),
                                         int(relu), _dp(out_scale), _dp(yq), yq.stride(0), _dp(partials),
                                         _stream_ptr(stream)), "pipe_expanded_conv2d_q8")


def pipe_lower_conv_input(geom: ConvGeom, xq_nhwc: torch.Tensor, rows: torch.Tensor, stream=None) -> None:
    """xq_nhwc: cuda int8 [N, H, W, C] contiguous; rows: cuda int8 [N*Ho*Wo, >= kh*kw*C] (last dim contiguous)."""
    assert xq_nhwc.is_contiguous() and xq_nhwc.dtype == torch.int8 and rows.dtype == torch.int8 and rows.stride(1) == 1
    _check(lib().pipe_lower_conv_input(C.byref(geom), _dp(xq_nhwc), _dp(rows), rows.stride(0), _stream_ptr(stream)),
           "pipe_lower_conv_input")


def pipe_ensemble_conv2d(desc: LayerDesc, geom: ConvGeom, blob: torch.Tensor, xq_m, sx_m, y_m, bias: torch.Tensor | None = None,
                         sum_branches: bool = False, partials: torch.Tensor | None = None, stream=None) -> None:
    """xq_m: M cuda int8 [N, H, W, C] contiguous tensors; y_m: M (or, summed, one) cuda float32 [N*Ho*Wo, O] tensors."""
    M = desc.num_branches
    assert len(xq_m) == M and len(sx_m) == M and len(y_m) >= (1 if sum_branches else M)
    assert all(t.is_contiguous() and t.dtype == torch.int8 for t in xq_m)
    PA = C.c_void_p * M
    xp = PA(*[_dp(t) for t in xq_m])
    sp = PA(*[_dp(t) for t in sx_m])
    yp = PA(*[(_dp(y_m[m]) if m < len(y_m) else None) for m in range(M)])
    _check(lib().pipe_ensemble_conv2d(C.byref(desc), C.byref(geom), _dp(blob), xp, sp, _dp(bias), yp, y_m[0].stride(0),
                                      1 if sum_branches else 0, _dp(partials), _stream_ptr(stream)), "pipe_ensemble_conv2d")


def pipe_ensemble_conv2d_q8(desc: LayerDesc, geom: ConvGeom, blob: torch.Tensor, xq_m, sx_m, out_scale_m, yq_m,
                            bias: torch.Tensor | None = None, relu: bool = True, partials: torch.Tensor | None = None,
                            stream=None) -> None:
    """Inner convolution of the M predictors: yq_m[m] (cuda int8 [N*Ho*Wo, O]) receives Q(sigma(y_m))."""
    M = desc.num_branches
    assert len(xq_m) == M and len(sx_m) == M and len(out_scale_m) == M and len(yq_m) == M
    assert all(t.is_contiguous() and t.dtype == torch.int8 for t in xq_m) and all(t.dtype == torch.int8 for t in yq_m)
    PA = C.c_void_p * M
    xp = PA(*[_dp(t) for t in xq_m])
    sp = PA(*[_dp(t) for t in sx_m])
    op = PA(*[_dp(t) for t in out_scale_m])
    yp = PA(*[_dp(t) for t in yq_m])
    _check(lib().pipe_ensemble_conv2d_q8(C.byref(desc), C.byref(geom), _dp(blob), xp, sp, _dp(bias), int(relu), op, yp,
                                         yq_m[0].stride(0), _dp(partials), _stream_ptr(stream)), "pipe_ensemble_conv2d_q8")


def pipe_ensemble_forward(desc: LayerDesc, blob: torch.Tensor, xq_m, sx_m, y_m, bias: torch.Tensor | None = None,
                          sum_branches: bool = False, partials: torch.Tensor | None = None, stream=None) -> None:
    """xq_m, sx_m, y_m: sequences of M cuda tensors (xq_m entries may be the same tensor)."""
    M = desc.num_branches
    assert len(xq_m) == M and len(sx_m) == M and len(y_m) >= (1 if sum_branches else M)
    T = xq_m[0].shape[0]
    ldxq = xq_m[0].stride(0) if T > 1 else max(xq_m[0].shape[1], xq_m[0].stride(0))
    ldy = y_m[0].stride(0) if T > 1 else max(y_m[0].shape[1], y_m[0].stride(0))
    PA = C.c_void_p * M
    xp = PA(*[_dp(t) for t in xq_m])
    sp = PA(*[_dp(t) for t in sx_m])
    yp = PA(*[(_dp(y_m[m]) if m < len(y_m) else None) for m in range(M)])
    _check(lib().pipe_ensemble_forward(C.byref(desc), _dp(blob), xp, T, ldxq, sp, _dp(bias), yp, ldy,
                                       1 if sum_branches else 0, _dp(partials), _stream_ptr(stream)),
           "pipe_ensemble_forward")


def pipe_ensemble_forward_q8(desc: LayerDesc, blob: torch.Tensor, xq_m, sx_m, out_scale_m, yq_m,
                             bias: torch.Tensor | None = None, relu: bool = True, partials: torch.Tensor | None = None,
                             stream=None) -> None:
    """Inner layer of the M predictors: yq_m[m] (cuda int8 [T, O]) receives Q(sigma(y_m)) with the static step
    out_scale_m[m] (cuda float32, one element); xq_m, sx_m as in pipe_ensemble_forward."""
    M = desc.num_branches
    assert len(xq_m) == M and len(sx_m) == M and len(out_scale_m) == M and len(yq_m) == M
    assert all(t.dtype == torch.int8 for t in yq_m)
    T = xq_m[0].shape[0]
    ldxq = xq_m[0].stride(0) if T > 1 else max(xq_m[0].shape[1], xq_m[0].stride(0))
    ldyq = yq_m[0].stride(0) if T > 1 else max(yq_m[0].shape[1], yq_m[0].stride(0))
    PA = C.c_void_p * M
    xp = PA(*[_dp(t) for t in xq_m])
    sp = PA(*[_dp(t) for t in sx_m])
    op = PA(*[_dp(t) for t in out_scale_m])
    yp = PA(*[_dp(t) for t in yq_m])
    _check(lib().pipe_ensemble_forward_q8(C.byref(desc), _dp(blob), xp, T, ldxq, sp, _dp(bias), int(relu), op, yp,
                                          ldyq, _dp(partials), _stream_ptr(stream)), "pipe_ensemble_forward_q8")


def pipe_diag_select_kernel(which: int) -> None:
    _check(lib().pipe_diag_select_kernel(which), "pipe_diag_select_kernel")


def pipe_diag_mma_i8_rate(n_cols: int, mma_per_cta: int, cta_pairs: bool = False, stream=None) -> float:
    """Queues the issue-rate probe of the integer tensor pipe; returns the integer operations of the launch."""
    ops = C.c_double(0.0)
    _check(lib().pipe_diag_mma_i8_rate(int(n_cols), int(mma_per_cta), 1 if cta_pairs else 0, C.byref(ops), _stream_ptr(stream)),
           "pipe_diag_mma_i8_rate")
    return float(ops.value)


def pipe_diag_bounded_wait(limit_cycles: int, stream=None) -> None:
    _check(lib().pipe_diag_bounded_wait(int(limit_cycles), _stream_ptr(stream)), "pipe_diag_bounded_wait")


def pipe_launch_count() -> int:
    return int(lib().pipe_launch_count())


def pipe_poll_status(stream=None) -> int:
    out = C.c_int32(0)
    _check(lib().pipe_poll_status(_stream_ptr(stream), C.byref(out)), "pipe_poll_status")
    return int(out.value)


def pipe_status_string(status: int) -> str:
    return lib().pipe_status_string(status).decode()


# ------------------------------------------------------------------------------------------------
# Convenience: device buffers for one layer (allocation is PyTorch's job, not the library's).
@dataclass
class ExpandedLayer:
    desc: LayerDesc
    layout: LayerLayout
    blob: torch.Tensor

    def section(self, off: int, nbytes: int) -> torch.Tensor:
        return self.blob[off:off + nbytes]

    def codes(self, k: int) -> torch.Tensor:
        n = self.layout.rows[k] * self.layout.canon_row_bytes
        return self.section(self.layout.codes_off[k], n).view(self.layout.rows[k], self.layout.canon_row_bytes)

    def kcodes(self, k: int) -> torch.Tensor:
        n = self.layout.rows[k] * self.layout.kernel_row_bytes
        return self.section(self.layout.kcodes_off[k], n).view(self.layout.rows[k], self.layout.kernel_row_bytes)

    def wcodes(self, k: int) -> torch.Tensor | None:
        """The int8 copy of order k as stored: [I_pad / 128, rows, 128] bytes (None without int8_copy)."""
        if not self.layout.wcodes_off[k]:
            return None
        ipad = (self.desc.in_features + 127) // 128 * 128
        n = self.layout.rows[k] * ipad
        return self.section(self.layout.wcodes_off[k], n).view(ipad // 128, self.layout.rows[k], 128)

    def scales(self, k: int) -> torch.Tensor:
        return self.section(self.layout.scales_off[k], self.layout.rows[k] * 4).view(torch.float32)

    def kept(self, k: int) -> torch.Tensor:
        return self.section(self.layout.kept_off[k], self.layout.kept_groups[k] * 4).view(torch.int32)

    def cum(self, k: int) -> torch.Tensor:
        return self.section(self.layout.cum_off[k], (self.layout.num_groups + 1) * 4).view(torch.int32)

    def decode_table(self, m: int) -> torch.Tensor | None:
        """Decode-unit table m (int32: n, b_0 .. b_n), or None when the cluster has none."""
        if self.layout.dec_off[m] == 0:
            return None
        return self.section(self.layout.dec_off[m], (self.layout.num_groups + 2) * 4).view(torch.int32)

    def block_records(self, m: int) -> torch.Tensor | None:
        """Block records of table m as bytes [rec_cap, BLOCK_RECORD_BYTES] (the first n of them are written), or None."""
        if self.layout.rec_off[m] == 0:
            return None
        return self.section(self.layout.rec_off[m], self.layout.rec_cap[m] * BLOCK_RECORD_BYTES).view(-1, BLOCK_RECORD_BYTES)

    def block_table(self, m: int) -> torch.Tensor | None:
        """Channel-block table m (int32: n, b_0 .. b_n), or None when the cluster has none."""
        if self.layout.blk_off[m] == 0:
            return None
        return self.section(self.layout.blk_off[m], (self.layout.blk_cap[m] + 2) * 4).view(torch.int32)


def last_kept_scales(layer: "ExpandedLayer"):
    """float32 host array [O]: the scale every output channel had at the last order that kept it (a device -> host
    read of the blob's scale sections and kept lists; no arithmetic)."""
    import numpy as np
    O, g = layer.desc.out_features, layer.desc.group_size
    out = np.zeros(O, np.float32)
    for k in range(layer.desc.num_orders):
        kept = layer.kept(k).cpu().numpy().astype(np.int64)
        ch = (kept[:, None] * g + np.arange(g)[None, :]).reshape(-1)
        out[ch] = layer.scales(k).cpu().numpy()
    return out


def alloc_bytes(nbytes: int, device="cuda") -> torch.Tensor:
    """uint8 device buffer whose start is aligned to BLOB_ALIGN."""
    raw = torch.empty(int(nbytes) + BLOB_ALIGN, dtype=torch.uint8, device=device)
    shift = (-raw.data_ptr()) % BLOB_ALIGN
    return raw[shift:shift + int(nbytes)]


def expand(desc: LayerDesc, W: torch.Tensor, stream=None) -> ExpandedLayer:
    lay = pipe_layout(desc)
    blob = alloc_bytes(lay.blob_bytes, W.device)
    ws = alloc_bytes(lay.expand_ws_bytes, W.device)
    pipe_expand_weights(desc, W, blob, ws, stream)
    return ExpandedLayer(desc, lay, blob)
