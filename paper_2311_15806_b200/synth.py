"""Seeded synthetic workloads shaped like the paper's ConvNet / BERT / LLM layers.

This module only draws random tensors and lowers a convolution input to GEMM rows; it
contains none of the method's arithmetic (no quantizer, no expansion, no selection), so
the CUDA library's tests and the CPU oracle can both take their inputs from it.

Streams: weights come from ``default_rng([seed, 0])`` in the fixed draw order
"base values -> per-row multipliers -> outlier positions -> outlier signs"; the
activations of ensemble branch ``m`` come from ``default_rng([seed, 1, m])`` in the order
"base values -> outlier channels".  Everything is cast to float32 at the end.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np


@dataclass(frozen=True)
class LayerSpec:
    name: str
    O: int                 # output features (rows of W)
    I: int                 # input features (reduction length)
    T: int                 # tokens (rows of x)
    bits: int              # weight bits: 8, 4 or 2 (ternary)
    K: int                 # expansion orders
    g: int                 # output channels per sparsity group
    gamma: float           # kept fraction of groups for orders >= 2
    M: int                 # ensemble branches
    seed: int
    w_dist: str            # "normal_rowmult", "student_t", "normal_outliers"
    w_scale: float
    w_param: tuple = ()
    x_dist: str = "normal"  # "normal", "relu_normal", "normal_chan_outliers"
    conv: tuple | None = None  # (N, H, W, C, kh, kw, pad) for an NHWC 3x3-style convolution

    def with_tokens(self, T: int) -> "LayerSpec":
        return replace(self, T=T)


def paper_workloads() -> dict[str, LayerSpec]:
    """The five configurations (two linears each for the FFN / MLP shaped ones)."""
    w = {}
    w["cfg1"] = LayerSpec("cfg1", 256, 256, 64, 8, 2, 8, 1.0, 1, 0, "normal_rowmult", 0.02, (0.5, 2.0))
    w["cfg2"] = LayerSpec("cfg2", 256, 2304, 32 * 56 * 56, 4, 3, 8, 0.25, 1, 1, "student_t", 0.02, (4.0,),
                          "relu_normal", (32, 56, 56, 256, 3, 3, 1))
    w["cfg3a"] = LayerSpec("cfg3a", 3072, 768, 4096, 4, 4, 8, 0.5, 2, 2, "normal_outliers", 0.02, (0.001, 10.0))
    w["cfg3b"] = LayerSpec("cfg3b", 768, 3072, 4096, 4, 4, 8, 0.5, 2, 2, "normal_outliers", 0.02, (0.001, 10.0))
    for T in (1, 16, 128, 1024, 4096):
        w[f"cfg4a_t{T}"] = LayerSpec(f"cfg4a_t{T}", 11008, 4096, T, 4, 4, 8, 0.5, 2, 3, "normal_rowmult", 0.02,
                                     (0.25, 4.0), "normal_chan_outliers")
        w[f"cfg4b_t{T}"] = LayerSpec(f"cfg4b_t{T}", 4096, 11008, T, 4, 4, 8, 0.5, 2, 3, "normal_rowmult", 0.02,
                                     (0.25, 4.0), "normal_chan_outliers")
    w["cfg5"] = LayerSpec("cfg5", 8192, 8192, 8192, 2, 8, 16, 0.25, 4, 4, "student_t", 0.015, (4.0,))
    return w


def scaled_down(spec: LayerSpec, O: int, I: int, T: int) -> LayerSpec:
    """Same distributions and quantization settings on a smaller shape (oracle-sized cases)."""
    return replace(spec, name=f"{spec.name}_small", O=O, I=I, T=T, conv=None)


def make_weights(spec: LayerSpec, second_layer: bool = False) -> np.ndarray:
    """float32 [O, I].  ``second_layer`` selects an independent stream for a layer that
    shares its seed with another one (the two linears of an FFN)."""
    rng = np.random.default_rng([spec.seed, 0, 1 if second_layer else 0])
    O, I = spec.O, spec.I
    if spec.w_dist == "normal_rowmult":
        W = rng.standard_normal((O, I), dtype=np.float32) * np.float32(spec.w_scale)
        lo, hi = spec.w_param
        mult = np.exp(rng.uniform(np.log(lo), np.log(hi), size=O)).astype(np.float32)
        W *= mult[:, None]
    elif spec.w_dist == "student_t":
        W = (rng.standard_t(spec.w_param[0], size=(O, I)) * spec.w_scale).astype(np.float32)
    elif spec.w_dist == "normal_outliers":
        W = rng.standard_normal((O, I), dtype=np.float32) * np.float32(spec.w_scale)
        frac, nsigma = spec.w_param
        n_out = int(round(frac * O * I))
        pos = rng.choice(O * I, size=n_out, replace=False)
        sign = rng.integers(0, 2, size=n_out) * 2 - 1
        W.reshape(-1)[pos] = (sign * nsigma * spec.w_scale).astype(np.float32)
    else:
        raise ValueError(spec.w_dist)
    return np.ascontiguousarray(W, dtype=np.float32)


def make_activations(spec: LayerSpec, branch: int = 0) -> np.ndarray:
    """float32 [T, I] GEMM rows; for a convolution spec use ``make_conv_input`` + ``im2col_rows``."""
    rng = np.random.default_rng([spec.seed, 1, branch])
    T, I = spec.T, spec.I
    x = rng.standard_normal((T, I), dtype=np.float32)
    if spec.x_dist == "relu_normal":
        np.maximum(x, 0, out=x)
    elif spec.x_dist == "normal_chan_outliers":
        n_ch = max(1, int(round(0.005 * I)))
        ch = rng.choice(I, size=n_ch, replace=False)
        x[:, ch] *= np.float32(20.0)
    elif spec.x_dist != "normal":
        raise ValueError(spec.x_dist)
    return x


def make_conv_input(spec: LayerSpec, branch: int = 0) -> np.ndarray:
    """float32 NHWC input of a convolution spec: ReLU(N(0,1))."""
    assert spec.conv is not None
    N, H, W_, C, _, _, _ = spec.conv
    rng = np.random.default_rng([spec.seed, 1, branch])
    x = rng.standard_normal((N, H, W_, C), dtype=np.float32)
    if spec.x_dist == "relu_normal":
        np.maximum(x, 0, out=x)
    return x


def im2col_rows(x_nhwc: np.ndarray, conv: tuple, rows: np.ndarray | None = None) -> np.ndarray:
    """Lower a stride-1 convolution input to GEMM rows.

    Row ``t = (n*H + h)*W + w`` holds, for every filter tap ``(dh, dw)`` in row-major
    order, the C channels of input pixel ``(n, h+dh-pad, w+dw-pad)`` (zeros outside the
    image), i.e. reduction index ``(dh*kw + dw)*C + c`` -- the order of a weight tensor
    ``[O, kh, kw, C]`` flattened to ``[O, kh*kw*C]``.  ``rows`` selects a subset of t.
    """
    N, H, W_, C, kh, kw, pad = conv
    if rows is None:
        rows = np.arange(N * H * W_)
    rows = np.asarray(rows, dtype=np.int64)
    n, rem = np.divmod(rows, H * W_)
    h, w = np.divmod(rem, W_)
    out = np.zeros((rows.shape[0], kh * kw * C), dtype=x_nhwc.dtype)
    for dh in range(kh):
        for dw in range(kw):
            hh, ww = h + dh - pad, w + dw - pad
            ok = (hh >= 0) & (hh < H) & (ww >= 0) & (ww < W_)
            tap = dh * kw + dw
            out[ok, tap * C:(tap + 1) * C] = x_nhwc[n[ok], hh[ok], ww[ok], :]
    return out


def sample_rows(T: int, count: int, tile: int, seed: int) -> np.ndarray:
    """Sorted token rows for sampled checks: first and last rows, both sides of every few
    tile boundaries, plus seeded random rows."""
    rng = np.random.default_rng([seed, 7])
    picks = {0, T - 1}
    for b in range(tile, T, max(tile, (T // 8 // tile) * tile or tile)):
        picks.update({b - 1, b})
    picks = {p for p in picks if 0 <= p < T}
    extra = max(0, count - len(picks))
    if extra:
        picks.update(int(v) for v in rng.choice(T, size=min(T, extra), replace=False))
    return np.array(sorted(picks), dtype=np.int64)
