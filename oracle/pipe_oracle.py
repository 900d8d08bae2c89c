"""ctypes front end of the CPU oracle (``pipe_oracle.c``).  TEST INFRASTRUCTURE.

Only the test-suite, the smoke check and the benchmark's CPU-baseline leg use this module;
the CUDA library never does.  ``build()`` compiles the C file with gcc into
``libpipe_oracle.so`` next to it; everything else marshals NumPy arrays.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pipe_oracle.c")
_SRC_EXT = os.path.join(_HERE, "pipe_oracle_ext.c")
_LIB = os.path.join(_HERE, "libpipe_oracle.so")

OK, ERR_ARG, ERR_NONFINITE, ERR_ACC_OVERFLOW = 0, 1, 2, 3


def build(force: bool = False) -> str:
    """Compile the oracle (plain C, -O2, OpenMP over rows, no contraction of a*b+c)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < max(os.path.getmtime(_SRC), os.path.getmtime(_SRC_EXT)):
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               "-fno-fast-math", "-Wall", "-o", _LIB, _SRC, _SRC_EXT, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        build()
        _lib = C.CDLL(_LIB)
        i32, i64, p = C.c_int32, C.c_int64, C.c_void_p
        _lib.pipe_oracle_threads.restype = C.c_int
        _lib.pipe_oracle_row_absmax.argtypes = [p, i64, i64, i64, p]
        _lib.pipe_oracle_select_groups.argtypes = [p, i32, i32, i32, p]
        _lib.pipe_oracle_expand.argtypes = [p, i64, i64, i64, C.c_int, C.c_int, i32, i32, p, p, p, p, p, p]
        _lib.pipe_oracle_pack.argtypes = [p, i64, i64, C.c_int, p]
        _lib.pipe_oracle_quantize_act.argtypes = [p, i64, i64, i64, p, p, i64, p]
        _lib.pipe_oracle_forward.argtypes = [p, i64, i64, i64, i64, C.c_int, i32, p, p, p, p, C.c_int, C.c_int,
                                             C.c_float, p, p, i64, p, p, p]
        _lib.pipe_oracle_ensemble.argtypes = [p, i64, i64, i64, C.c_int, i32, p, p, p, p, C.c_int, p, p, p,
                                              C.c_int, p, p]
        _lib.pipe_oracle_balanced_split.argtypes = [C.c_int, C.c_int, p]
        _lib.pipe_oracle_keep_groups.argtypes = [i32, C.c_double]
        _lib.pipe_oracle_keep_groups.restype = i32
        # pipe_oracle_ext.c
        _lib.pipe_oracle_select_groups_ex.argtypes = [p, i64, i64, i32, i32, C.c_int, p, p]
        _lib.pipe_oracle_expand_ex.argtypes = [p, i64, i64, i64, C.c_int, C.c_int, i32, i32, C.c_int, i64, p, p, p, p, p]
        _lib.pipe_oracle_container_bits.argtypes = [C.c_int]
        _lib.pipe_oracle_pack_ex.argtypes = [p, i64, i64, C.c_int, p]
        _lib.pipe_oracle_quantize_act_ex.argtypes = [p, i64, i64, i64, C.c_int, C.c_int, p, p, p, i64, p, p]
        _lib.pipe_oracle_forward_zp.argtypes = [p, i64, i64, i64, i64, C.c_int, i32, p, p, p, p, C.c_int, C.c_int,
                                                C.c_float, i32, p, p, i64, p, p, p, p]
        _lib.pipe_oracle_activation.argtypes = [p, i64, C.c_int, p]
    return _lib


def threads() -> int:
    return int(lib().pipe_oracle_threads())


class OracleError(RuntimeError):
    def __init__(self, code: int):
        super().__init__(f"oracle returned status {code}")
        self.code = code


def _check(rc: int) -> None:
    if rc != OK:
        raise OracleError(rc)


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


@dataclass
class Expansion:
    """Output of the expansion: compacted per-order codes/scales and kept-group lists."""
    O: int
    I: int
    bits: int
    K: int
    g: int
    n_keep: int
    codes: np.ndarray        # int8 [R_total, I]
    scales: np.ndarray       # float32 [R_total]
    kept: np.ndarray         # int32 [K, G]
    kept_count: np.ndarray   # int32 [K]
    residual: np.ndarray     # float32 [O, I]
    absmax: np.ndarray       # float32 [K, O]

    @property
    def G(self) -> int:
        return self.O // self.g

    def rows(self, k: int) -> int:
        return int(self.kept_count[k]) * self.g

    def row_off(self, k: int) -> int:
        return int(sum(self.rows(j) for j in range(k)))

    @property
    def R_total(self) -> int:
        return self.row_off(self.K)

    def order_codes(self, k: int) -> np.ndarray:
        return self.codes[self.row_off(k):self.row_off(k) + self.rows(k)]

    def order_scales(self, k: int) -> np.ndarray:
        return self.scales[self.row_off(k):self.row_off(k) + self.rows(k)]

    def order_kept(self, k: int) -> np.ndarray:
        return self.kept[k, :int(self.kept_count[k])]

    def order_channels(self, k: int) -> np.ndarray:
        """Output channel of every compacted row of order k."""
        kg = self.order_kept(k).astype(np.int64)
        return (kg[:, None] * self.g + np.arange(self.g)[None, :]).reshape(-1)

    def packed(self, k: int) -> np.ndarray:
        if self.bits in (3, 6):
            return pack_ex(self.order_codes(k), self.bits)
        return pack(self.order_codes(k), self.bits)


def row_absmax(r: np.ndarray) -> np.ndarray:
    r = _c(r, np.float32)
    a = np.empty(r.shape[0], np.float32)
    _check(lib().pipe_oracle_row_absmax(_ptr(r), r.shape[0], r.shape[1], r.shape[1], _ptr(a)))
    return a


def select_groups(a: np.ndarray, g: int, n_keep: int) -> np.ndarray:
    a = _c(a, np.float32)
    G = a.shape[0] // g
    out = np.empty(n_keep, np.int32)
    _check(lib().pipe_oracle_select_groups(_ptr(a), G, g, n_keep, _ptr(out)))
    return out


def expand(W: np.ndarray, bits: int, K: int, g: int, n_keep: int) -> Expansion:
    W = _c(W, np.float32)
    O, I = W.shape
    G = O // g
    R_max = O + (K - 1) * n_keep * g
    codes = np.zeros((R_max, I), np.int8)
    scales = np.zeros(R_max, np.float32)
    kept = np.full((K, G), -1, np.int32)
    kept_count = np.zeros(K, np.int32)
    residual = np.empty((O, I), np.float32)
    absmax = np.empty((K, O), np.float32)
    _check(lib().pipe_oracle_expand(_ptr(W), O, I, I, bits, K, g, n_keep, _ptr(codes), _ptr(scales), _ptr(kept),
                                    _ptr(kept_count), _ptr(residual), _ptr(absmax)))
    R = int(kept_count.astype(np.int64).sum()) * g
    return Expansion(O, I, bits, K, g, n_keep, codes[:R], scales[:R], kept, kept_count, residual, absmax)


def pack(codes: np.ndarray, bits: int) -> np.ndarray:
    codes = _c(codes, np.int8)
    rows, I = codes.shape
    per = 8 // bits
    out = np.empty((rows, (I + per - 1) // per), np.uint8)
    _check(lib().pipe_oracle_pack(_ptr(codes), rows, I, bits, _ptr(out)))
    return out


def quantize_act(x: np.ndarray, static_scale: float | None = None):
    x = _c(x, np.float32)
    T, I = x.shape
    xq = np.empty((T, I), np.int8)
    sx = np.zeros(1, np.float32)
    ss = None if static_scale is None else np.array([static_scale], np.float32)
    _check(lib().pipe_oracle_quantize_act(_ptr(x), T, I, I, _ptr(ss), _ptr(xq), I, _ptr(sx)))
    return xq, np.float32(sx[0])


# ---- variants beside the main setting (pipe_oracle_ext.c) --------------------------------------------------
SCORE_MAXABS, SCORE_L2 = 0, 1
ACT_IDENTITY, ACT_RELU, ACT_SILU, ACT_GELU, ACT_SIGMOID = 0, 1, 2, 3, 4


def container_bits(bits: int) -> int:
    return int(lib().pipe_oracle_container_bits(bits))


def select_groups_ex(r: np.ndarray, g: int, n_keep: int, score_mode: int):
    """Kept groups (ascending) and the scores [G] (binary64) of the residual r [O, I]."""
    r = _c(r, np.float32)
    O, I = r.shape
    out = np.empty(n_keep, np.int32)
    score = np.empty(O // g, np.float64)
    _check(lib().pipe_oracle_select_groups_ex(_ptr(r), O, I, g, n_keep, score_mode, _ptr(out), _ptr(score)))
    return out, score


def expand_ex(W: np.ndarray, bits: int, K: int, g: int, n_keep: int, score_mode: int = 0, elem_keep: int = 0) -> Expansion:
    """The expansion for b in {2, 3, 4, 6, 8}, either group score, optionally the unstructured mask."""
    W = _c(W, np.float32)
    O, I = W.shape
    G = O // g
    R_max = O + (K - 1) * n_keep * g
    codes = np.zeros((R_max, I), np.int8)
    scales = np.zeros(R_max, np.float32)
    kept = np.full((K, G), -1, np.int32)
    kept_count = np.zeros(K, np.int32)
    residual = np.empty((O, I), np.float32)
    _check(lib().pipe_oracle_expand_ex(_ptr(W), O, I, I, bits, K, g, n_keep, score_mode, elem_keep, _ptr(codes), _ptr(scales),
                                       _ptr(kept), _ptr(kept_count), _ptr(residual)))
    R = int(kept_count.astype(np.int64).sum()) * g
    return Expansion(O, I, bits, K, g, n_keep, codes[:R], scales[:R], kept, kept_count, residual, np.zeros((K, O), np.float32))


def pack_ex(codes: np.ndarray, bits: int) -> np.ndarray:
    codes = _c(codes, np.int8)
    rows, I = codes.shape
    per = 8 // container_bits(bits)
    out = np.empty((rows, (I + per - 1) // per), np.uint8)
    _check(lib().pipe_oracle_pack_ex(_ptr(codes), rows, I, bits, _ptr(out)))
    return out


def quantize_act_ex(x: np.ndarray, act_bits: int = 8, asymmetric: bool = False, static_scale: float | None = None,
                    static_range=None):
    """Returns (codes int8 [T, I], lambda_x, zero point)."""
    x = _c(x, np.float32)
    T, I = x.shape
    xq = np.empty((T, I), np.int8)
    sx = np.zeros(1, np.float32)
    zp = np.zeros(1, np.int32)
    ss = None if static_scale is None else np.array([static_scale], np.float32)
    sr = None if static_range is None else np.array(static_range, np.float32)
    _check(lib().pipe_oracle_quantize_act_ex(_ptr(x), T, I, I, act_bits, int(bool(asymmetric)), _ptr(ss), _ptr(sr), _ptr(xq), I,
                                             _ptr(sx), _ptr(zp)))
    return xq, np.float32(sx[0]), int(zp[0])


def forward_zp(e: Expansion, xq: np.ndarray, sx, zero_point: int, k_begin: int = 0, k_end: int | None = None,
               bias: np.ndarray | None = None):
    """`forward` on asymmetric codes: the contraction runs on (c - zero_point).  Returns (Forward, rowsum int64 [R_total])."""
    xq = _c(xq, np.int8)
    T, I = xq.shape
    k_end = e.K if k_end is None else k_end
    y = np.empty((T, e.O), np.float32)
    y64 = np.empty((T, e.O), np.float64)
    yabs = np.empty((T, e.O), np.float64)
    partials = np.zeros((T, e.R_total), np.int32)
    rowsum = np.zeros(e.R_total, np.int64)
    b = None if bias is None else _c(bias, np.float32)
    _check(lib().pipe_oracle_forward_zp(_ptr(xq), T, I, I, e.O, e.K, e.g, _ptr(e.codes), _ptr(e.scales), _ptr(e.kept),
                                        _ptr(e.kept_count), k_begin, k_end, C.c_float(float(sx)), int(zero_point), _ptr(b),
                                        _ptr(y), e.O, _ptr(y64), _ptr(yabs), _ptr(partials), _ptr(rowsum)))
    return Forward(y, y64, yabs, partials), rowsum


def activation(v: np.ndarray, kind: int) -> np.ndarray:
    v = _c(v, np.float32)
    out = np.empty_like(v)
    _check(lib().pipe_oracle_activation(_ptr(v), v.size, kind, _ptr(out)))
    return out


def forward_requantized(e: "Expansion", xq: np.ndarray, sx, out_scale: float, k_begin: int = 0, k_end: int | None = None,
                        bias: np.ndarray | None = None, relu: bool = True) -> np.ndarray:
    """One inner layer of an ensemble branch (Sec. 3.2; Appendix B, the predictors g and h): the branch's
    cluster of orders on its own input, the activation function, then the next layer's input quantizer Q
    with a static scale.  Nothing new is computed here: it is `forward`, a ReLU, and `quantize_act`."""
    y = forward(e, xq, sx, k_begin, k_end, bias).y
    if relu:
        y = np.maximum(y, np.float32(0))
    return quantize_act(y, static_scale=out_scale)[0]


@dataclass
class Forward:
    y: np.ndarray          # float32 [T, O]
    y64: np.ndarray        # float64 [T, O]  same sum in binary64
    yabs: np.ndarray       # float64 [T, O]  sum of |terms|
    partials: np.ndarray   # int32 [T, R_total] (only the cluster's columns written)


def forward(e: Expansion, xq: np.ndarray, sx, k_begin: int = 0, k_end: int | None = None,
            bias: np.ndarray | None = None) -> Forward:
    xq = _c(xq, np.int8)
    T, I = xq.shape
    assert I == e.I
    k_end = e.K if k_end is None else k_end
    y = np.empty((T, e.O), np.float32)
    y64 = np.empty((T, e.O), np.float64)
    yabs = np.empty((T, e.O), np.float64)
    partials = np.zeros((T, e.R_total), np.int32)
    b = None if bias is None else _c(bias, np.float32)
    _check(lib().pipe_oracle_forward(_ptr(xq), T, I, I, e.O, e.K, e.g, _ptr(e.codes), _ptr(e.scales), _ptr(e.kept),
                                     _ptr(e.kept_count), k_begin, k_end, C.c_float(float(sx)), _ptr(b), _ptr(y),
                                     e.O, _ptr(y64), _ptr(yabs), _ptr(partials)))
    return Forward(y, y64, yabs, partials)


def ensemble(e: Expansion, xq_m: np.ndarray, sx_m, branch_orders, bias=None, sum_branches=False):
    """xq_m: [M, T, I] int8; returns (y [M,T,O] or [T,O], partials [T, R_total])."""
    xq_m = _c(xq_m, np.int8)
    M, T, I = xq_m.shape
    bo = _c(branch_orders, np.int32)
    sx = _c(sx_m, np.float32)
    y = np.empty((T, e.O) if sum_branches else (M, T, e.O), np.float32)
    partials = np.zeros((T, e.R_total), np.int32)
    b = None if bias is None else _c(bias, np.float32)
    _check(lib().pipe_oracle_ensemble(_ptr(xq_m), T, I, e.O, e.K, e.g, _ptr(e.codes), _ptr(e.scales), _ptr(e.kept),
                                      _ptr(e.kept_count), M, _ptr(bo), _ptr(sx), _ptr(b), int(bool(sum_branches)),
                                      _ptr(y), _ptr(partials)))
    return y, partials


def balanced_split(K: int, M: int) -> np.ndarray:
    out = np.zeros(M, np.int32)
    _check(lib().pipe_oracle_balanced_split(K, M, _ptr(out)))
    return out


def keep_groups(G: int, gamma: float) -> int:
    return int(lib().pipe_oracle_keep_groups(G, float(gamma)))


# ---- Appendix H (operation head-count) and the budget of Sec. 3.1 / 4.3: closed forms, written out
def bit_ops_original(d: int, D: int, n_i: int, n_o: int, s: int) -> float:
    """O_original = D^2 * d^2 n_i n_o / s^2 * 32 log 32 (Appendix H); log to base 2."""
    import math
    return D ** 2 * (d ** 2 * n_i * n_o / s ** 2) * 32.0 * math.log2(32.0)


def bit_ops_expanded(d: int, D: int, n_i: int, n_o: int, s: int, bits: int, orders: float) -> float:
    """O_R(k) = D^2 [ (n_i + n_o / s^2) 32 log 32 + k d^2 n_i n_o / s^2 b log b ] (Appendix H)."""
    import math
    return D ** 2 * ((n_i + n_o / s ** 2) * 32.0 * math.log2(32.0)
                     + orders * (d ** 2 * n_i * n_o / s ** 2) * bits * math.log2(bits))


def bound_network(s, u) -> float:
    """Appendix C, first theorem: U = prod_{l=1..L} (sum_{i<=l} s_i u_i + 1) - 1, written out."""
    U, acc = 1.0, 0.0
    for sl, ul in zip(s, u):
        acc += sl * ul
        U *= acc + 1.0
    return U - 1.0


def bound_step_dense(bits: int, K: int, first_scale_max: float) -> float:
    """u^(K) of Lemma B.1 / Appendix C: (1 / (2^(b-1) - 1))^(K-1) * lambda / 2."""
    return (1.0 / (2 ** (bits - 1) - 1)) ** (K - 1) * first_scale_max / 2.0


def choose_expansion(d, D, n_i, n_o, s, bits, budget, max_orders, min_gamma, num_branches):
    """Sec. 3.1 / App. A / App. H: the number of full orders the budget pays for, then the largest K whose kept
    fraction stays >= min_gamma; balanced predictors.  Returns (K, gamma, [K_m])."""
    import math
    rescale = bit_ops_expanded(d, D, n_i, n_o, s, bits, 0.0)
    one = bit_ops_expanded(d, D, n_i, n_o, s, bits, 1.0) - rescale
    beta = min((budget - rescale) / one, float(max_orders))
    K = max(1, min(max_orders, 1 + int(math.floor((beta - 1.0) / min_gamma + 1e-9))))
    gamma = 1.0 if K == 1 else min(1.0, (beta - 1.0) / (K - 1))
    M = min(num_branches, K)
    return K, gamma, [int(v) for v in balanced_split(K, M)]


def budget_of(K: int, gamma: float) -> float:
    """Full orders a group-sparse expansion costs: order 1 dense, K - 1 orders at kept fraction gamma."""
    return 1.0 + (K - 1) * gamma
