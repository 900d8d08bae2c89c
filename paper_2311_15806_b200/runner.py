"""One expanded layer on one GPU: device buffers plus the sequence of C-ABI calls of a step.

A step is the whole hot path on one batch: expand the fp32 weights, quantize the activations
of every ensemble branch, run the (grouped) expanded GEMM.  Used by the benchmark, the smoke
check and the full-size parity tests, so that what is timed is what is tested.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B
from . import synth


class LayerRunner:
    def __init__(self, spec: synth.LayerSpec, device="cuda", distinct_inputs: bool = True, second_layer: bool = False,
                 implicit_conv: bool = True, int8_copy: bool = False):
        self.spec = spec
        self.device = torch.device(device)
        G = spec.O // spec.g
        self.n_keep = B.pipe_keep_groups_from_gamma(G, spec.gamma)
        # int8_copy: the blob also keeps the codes as int8 in the tensor-core operand layout (pipe_layer_desc.int8_copy)
        self.desc = B.make_desc(spec.O, spec.I, spec.bits, spec.K, spec.g, self.n_keep, spec.M, int8_copy=int8_copy)
        self.layout = B.pipe_layout(self.desc)
        self.second_layer = second_layer
        # a convolution workload runs as implicit GEMM on the NHWC tensor when the library takes its shape
        self.geom = None
        if spec.conv is not None and implicit_conv:
            N, H, W_, C, kh, kw, pad = spec.conv
            if C % 128 == 0 and H % 8 == 0 and W_ % 8 == 0 and spec.M == 1:
                g = B.ConvGeom()
                g.batch, g.height, g.width, g.channels = N, H, W_, C
                g.kernel_h, g.kernel_w, g.pad_h, g.pad_w = kh, kw, pad, pad
                self.geom = g
        self.M = spec.M
        self.distinct_inputs = distinct_inputs and spec.M > 1
        self.blob = B.alloc_bytes(self.layout.blob_bytes, self.device)
        self.expand_ws = B.alloc_bytes(self.layout.expand_ws_bytes, self.device)
        self.quant_ws = [B.alloc_bytes(256, self.device) for _ in range(self.M)]
        self.W = None
        self.x = []      # per distinct input: float32 [T, I]
        self.xq = []
        self.sx = []
        self.y = []
        self.layer = B.ExpandedLayer(self.desc, self.layout, self.blob)

    # ---- inputs -------------------------------------------------------------------------------
    def host_weights(self) -> np.ndarray:
        return synth.make_weights(self.spec, self.second_layer)

    def host_inputs(self) -> list[np.ndarray]:
        """float32 [T, I] GEMM rows per distinct input (a convolution is lowered with im2col)."""
        n = self.M if self.distinct_inputs else 1
        out = []
        for m in range(n):
            if self.spec.conv is not None:
                out.append(None)  # too large to lower on the host; see load_inputs
            else:
                out.append(synth.make_activations(self.spec, m))
        return out

    def load(self, W: np.ndarray | None = None, xs: list | None = None) -> None:
        spec = self.spec
        W = self.host_weights() if W is None else W
        self.W = torch.from_numpy(W).to(self.device)
        n = self.M if self.distinct_inputs else 1
        self.x = []
        for m in range(n):
            if xs is not None and xs[m] is not None:
                self.x.append(torch.from_numpy(xs[m]).to(self.device))
            elif spec.conv is not None and self.geom is not None:
                N, H, W_, C = spec.conv[:4]
                self.x.append(torch.from_numpy(synth.make_conv_input(spec, m)).to(self.device).view(N * H * W_, C))
            elif spec.conv is not None:
                self.x.append(self._lower_conv_on_device(synth.make_conv_input(spec, m)))
            else:
                self.x.append(torch.from_numpy(synth.make_activations(spec, m)).to(self.device))
        T = self.x[0].shape[0]
        self.T = T
        self.xq = [torch.empty(tuple(self.x[0].shape), dtype=torch.int8, device=self.device) for _ in range(n)]
        self.sx = [torch.zeros(1, dtype=torch.float32, device=self.device) for _ in range(n)]
        self.y = [torch.empty((T, spec.O), dtype=torch.float32, device=self.device) for _ in range(self.M)]

    def _lower_conv_on_device(self, x_nhwc: np.ndarray) -> torch.Tensor:
        """im2col by index arithmetic on the device (input preparation, same row order as
        synth.im2col_rows): [N,H,W,C] -> [N*H*W, kh*kw*C] with a zero halo."""
        N, H, W_, C, kh, kw, pad = self.spec.conv
        x = torch.from_numpy(x_nhwc).to(self.device)
        xp = torch.zeros((N, H + 2 * pad, W_ + 2 * pad, C), dtype=x.dtype, device=self.device)
        xp[:, pad:pad + H, pad:pad + W_, :] = x
        out = torch.empty((N * H * W_, kh * kw * C), dtype=x.dtype, device=self.device)
        o4 = out.view(N, H, W_, kh * kw * C)
        for dh in range(kh):
            for dw in range(kw):
                tap = dh * kw + dw
                o4[..., tap * C:(tap + 1) * C] = xp[:, dh:dh + H, dw:dw + W_, :]
        return out

    # ---- the hot path -------------------------------------------------------------------------
    def expand(self) -> None:
        B.pipe_expand_weights(self.desc, self.W, self.blob, self.expand_ws)

    def quantize(self) -> None:
        for m in range(len(self.x)):
            B.pipe_quantize_act(self.x[m], self.xq[m], self.sx[m], self.quant_ws[m])

    def forward(self, partials: torch.Tensor | None = None, blob: torch.Tensor | None = None) -> None:
        blob = self.blob if blob is None else blob
        if self.geom is not None:
            N, H, W_, C = self.spec.conv[:4]
            B.pipe_expanded_conv2d(self.desc, self.geom, blob, self.xq[0].view(N, H, W_, C), self.sx[0], self.y[0], None,
                                   partials)
        elif self.M == 1:
            B.pipe_expanded_linear(self.desc, blob, self.xq[0], self.sx[0], self.y[0], None, partials)
        else:
            n = len(self.xq)
            xq = [self.xq[m if n > 1 else 0] for m in range(self.M)]
            sx = [self.sx[m if n > 1 else 0] for m in range(self.M)]
            B.pipe_ensemble_forward(self.desc, blob, xq, sx, self.y, None, False, partials)

    def forward_q8(self, out_scale: list, relu: bool = True, blob: torch.Tensor | None = None) -> list:
        """The layer as an inner layer of the predictors: int8 outputs Q(sigma(y_m)) with the static steps
        ``out_scale`` (M one-element cuda float32 tensors); no fp32 output is written.  Returns the M outputs."""
        blob = self.blob if blob is None else blob
        if not hasattr(self, "yq"):
            self.yq = [torch.empty(tuple(y.shape), dtype=torch.int8, device=self.device) for y in self.y]
        if self.geom is not None:
            N, H, W_, C = self.spec.conv[:4]
            B.pipe_expanded_conv2d_q8(self.desc, self.geom, blob, self.xq[0].view(N, H, W_, C), self.sx[0], out_scale[0],
                                      self.yq[0], None, relu)
            return self.yq
        n = len(self.xq)
        xq = [self.xq[m if n > 1 else 0] for m in range(self.M)]
        sx = [self.sx[m if n > 1 else 0] for m in range(self.M)]
        B.pipe_ensemble_forward_q8(self.desc, blob, xq, sx, out_scale, self.yq, None, relu)
        return self.yq

    def blob_copies(self, min_total_bytes: int) -> list:
        """The expanded blob plus enough byte copies of it that together they exceed
        ``min_total_bytes`` (for timing loops that must not re-read weights from L2)."""
        n = max(1, -(-int(min_total_bytes) // int(self.layout.blob_bytes)))
        out = [self.blob]
        for _ in range(n - 1):
            c = B.alloc_bytes(self.layout.blob_bytes, self.device)
            c.copy_(self.blob)
            out.append(c)
        return out

    def step(self) -> None:
        self.expand()
        self.quantize()
        self.forward()

    # ---- bookkeeping ----------------------------------------------------------------------------
    @property
    def total_rows(self) -> int:
        return int(self.layout.total_rows)

    def macs_per_token(self) -> int:
        """Multiply-accumulates of the contraction per token: I * sum_k rows_k (kept rows only)."""
        return self.spec.I * self.total_rows

    def forward_bytes(self) -> int:
        """Algorithmic bytes of one forward call: streamed codes + scales + xq + fp32 outputs."""
        lay, s = self.layout, self.spec
        row_bytes = lay.kernel_row_bytes
        if self.desc.int8_copy and self.T > 16:      # the kernels for more than 16 tokens read the int8 copy instead
            row_bytes = (s.I + 127) // 128 * 128
        codes = sum(lay.rows[k] * row_bytes for k in range(s.K))
        scales = 4 * self.total_rows + 4 * (lay.num_groups + 1) * s.K
        return codes + scales + sum(x.numel() for x in self.xq) + 4 * self.M * self.T * s.O

    def expand_bytes(self) -> int:
        """Algorithmic bytes of the expansion: every processed row is read and (except at the last
        order) written as fp32 residual, plus both code layouts written once."""
        lay, s = self.layout, self.spec
        b = 4 * s.O * s.I  # order-1 absmax pass
        for k in range(s.K):
            b += 4 * lay.rows[k] * s.I * (2 if k + 1 < s.K else 1)
            b += lay.rows[k] * (lay.canon_row_bytes + lay.kernel_row_bytes)
            if self.desc.int8_copy:
                b += lay.rows[k] * ((s.I + 127) // 128 * 128)
        return b

    def quantize_bytes(self) -> int:
        """absmax pass reads fp32 once, quantize pass reads it again and writes int8."""
        return sum(x.numel() for x in self.x) * (4 + 4 + 1)
