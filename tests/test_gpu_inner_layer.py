"""Inner layers of the ensemble (Sec. 3.2, Fig. 2; Appendix B, Eq. 9 with its activation function): the fused
epilogue sigma -> Q of pipe_ensemble_forward_q8 against the oracle's composition forward -> ReLU -> quantizer,
bit for bit, and a two-layer chain of predictors whose outputs meet only after the last layer."""
import numpy as np
import pytest
import torch

from paper_2311_15806_b200 import binding as B
from tests import gpu_harness as H

pytestmark = pytest.mark.gpu

KERNELS = [B.KERNEL_REFERENCE, B.KERNEL_TCGEN05, B.KERNEL_TCGEN05_PAIR, B.KERNEL_STREAM, B.KERNEL_DECODE_TC, B.KERNEL_AUTO]


@pytest.fixture(scope="module", autouse=True)
def _built():
    H.ensure_built()


def _w(rng, O, I, heavy=False):
    W = (rng.standard_t(4, size=(O, I)) if heavy else rng.standard_normal((O, I))) * 0.02
    W *= np.exp(rng.uniform(np.log(0.25), np.log(4.0), size=(O, 1)))
    return W.astype(np.float32)


INNER_CASES = [
    # O,   I,    T,  bits, K, g, n_keep, M, relu, pitch_extra
    (192, 1000, 150, 4, 4, 8, 12, 2, True, 0),
    (128, 328, 33, 2, 8, 16, 2, 4, True, 3),       # rows of the output not word aligned
    (264, 512, 16, 4, 4, 8, 17, 2, False, 0),      # decode sizes, no activation function
    (264, 512, 3, 4, 4, 8, 17, 2, True, 1),
    (256, 384, 9, 8, 2, 8, 16, 1, True, 0),
    (304, 2304, 131, 4, 3, 8, 19, 1, False, 4),
    (200, 144, 260, 8, 3, 8, 5, 3, True, 0),
    (512, 272, 1000, 2, 8, 16, 8, 4, True, 0),     # two token tiles per CTA tile
]


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("O,I,T,bits,K,g,n_keep,M,relu,pitch_extra", INNER_CASES)
def test_requantized_inner_layer_matches_oracle(oracle, kernel, O, I, T, bits, K, g, n_keep, M, relu, pitch_extra):
    rng = np.random.default_rng(7 * O + I + 11 * T)
    W = _w(rng, O, I, heavy=(bits == 2))
    bias = rng.standard_normal(O).astype(np.float32) * 0.1
    e = oracle.expand(W, bits, K, g, n_keep)
    d = H.desc_of(O, I, bits, K, g, n_keep, M)
    layer = H.gpu_expand(d, W)
    split = [layer.layout.branch_orders[m] for m in range(M)]
    xs = [(rng.standard_normal((T, I)) * (1 + m)).astype(np.float32) for m in range(M)]
    q = [H.gpu_quantize(x) for x in xs]
    qo = [oracle.quantize_act(x) for x in xs]

    # the step of every predictor: calibrated on the oracle's own fp32 output so that a few percent of the
    # values clamp (a static step does not follow the batch's maximum)
    steps, want = [], []
    k0 = 0
    want_part = np.zeros((T, e.R_total), np.int32)
    for m in range(M):
        b = bias if m == 0 else None
        fm = oracle.forward(e, qo[m][0], qo[m][1], k0, k0 + split[m], bias=b)
        a = np.maximum(fm.y, 0) if relu else fm.y
        s = float(np.float32(np.quantile(np.abs(a), 0.97) / 127 + 1e-12))
        steps.append(s)
        want.append(oracle.forward_requantized(e, qo[m][0], qo[m][1], s, k0, k0 + split[m], bias=b, relu=relu))
        lo, hi = e.row_off(k0), e.row_off(k0 + split[m])
        want_part[:, lo:hi] = fm.partials[:, lo:hi]
        k0 += split[m]
    try:
        got, part = H.gpu_ensemble_q8(layer, [a for a, _ in q], [b for _, b in q], steps, bias, relu=relu, kernel=kernel,
                                      pitch_extra=pitch_extra)
    except B.PipeError as ex:
        if ex.status == B.PIPE_ERR_UNSUPPORTED and kernel != B.KERNEL_AUTO:
            pytest.skip("this kernel does not take this shape (the automatic choice falls back)")
        raise
    assert B.pipe_poll_status() == B.PIPE_OK
    for m in range(M):
        np.testing.assert_array_equal(got[m], want[m], err_msg=f"predictor {m}")
        assert np.abs(want[m]).max() == 127     # the case does clamp
        if relu:
            assert want[m].min() == 0
    np.testing.assert_array_equal(part, want_part)


@pytest.mark.parametrize("kernel", KERNELS)
def test_requantization_at_rounding_boundaries(oracle, kernel):
    """Weights, steps and inputs are powers of two times integers, so every fp32 output is exact and many
    quotients y / s fall exactly half way between two codes: ties must go to the even code on both sides."""
    rng = np.random.default_rng(5)
    O, I, T = 128, 256, 96 if kernel not in (B.KERNEL_STREAM, B.KERNEL_DECODE_TC) else 16
    qw = rng.integers(-7, 8, size=(O, I))
    qw[:, 0] = 7                                   # every row spans the full 4-bit range: its scale is 2^-6 exactly
    W = (qw * 2.0 ** -6).astype(np.float32)
    e = oracle.expand(W, 4, 1, 8, O // 8)
    assert (e.scales == np.float32(2.0 ** -6)).all()
    d = H.desc_of(O, I, 4, 1, 8, O // 8, 1)
    layer = H.gpu_expand(d, W)
    xq = rng.integers(-3, 4, size=(T, I)).astype(np.int8)
    sx = np.float32(2.0 ** -4)
    s_out = 2.0 ** -7                              # y / s_out = acc / 8: one accumulator in eight is a tie
    f = oracle.forward(e, xq, sx)
    quot = f.partials[:, :O].astype(np.int64)
    assert ((quot % 8) == 4).sum() > 100
    want = oracle.forward_requantized(e, xq, sx, s_out, relu=False)
    # the definition, in integers: ties to even of acc / 8
    np.testing.assert_array_equal(want, np.clip(np.rint(quot / 8.0), -127, 127).astype(np.int8))
    try:
        got, _ = H.gpu_ensemble_q8(layer, [torch.from_numpy(xq).cuda()], [torch.tensor([sx], device="cuda")], [s_out],
                                   relu=False, kernel=kernel)
    except B.PipeError as ex:
        if ex.status == B.PIPE_ERR_UNSUPPORTED and kernel != B.KERNEL_AUTO:
            pytest.skip("this kernel does not take this shape")
        raise
    np.testing.assert_array_equal(got[0], want)


def test_requantization_next_to_rounding_boundaries(oracle):
    """Steps chosen so that one output's quotient y / s lies within a few units in the last place of n + 1/2:
    the tensor-core epilogue estimates the quotient with a reciprocal and must still give the code of the IEEE
    quotient, on whichever side of the boundary that falls."""
    rng = np.random.default_rng(23)
    O, I, T, bits, K, g, n_keep = 256, 512, 200, 4, 3, 8, 12
    W = _w(rng, O, I)
    e = oracle.expand(W, bits, K, g, n_keep)
    layer = H.gpu_expand(H.desc_of(O, I, bits, K, g, n_keep, 1), W)
    x = rng.standard_normal((T, I)).astype(np.float32)
    xq, sx = H.gpu_quantize(x)
    xq_o, sx_o = oracle.quantize_act(x)
    y = oracle.forward(e, xq_o, sx_o).y
    near = 0
    for trial in range(24):
        t, o = rng.integers(T), rng.integers(O)
        n = int(rng.integers(3, 120))
        s = np.float32(abs(y[t, o]) / np.float32(n + 0.5))
        if trial % 3:
            s = np.nextafter(s, np.float32(np.inf if trial % 3 == 1 else 0))   # one step above / below as well
        quot = y.astype(np.float64) / float(s)
        frac = np.abs(quot - np.floor(quot) - 0.5)
        near += int((frac < np.abs(quot) * 2.0 ** -21).sum())
        want = oracle.forward_requantized(e, xq_o, sx_o, float(s), relu=False)
        got, _ = H.gpu_ensemble_q8(layer, [xq], [sx], [float(s)], relu=False, kernel=B.KERNEL_TCGEN05, want_partials=False)
        np.testing.assert_array_equal(got[0], want, err_msg=f"trial {trial}, step {s}")
    assert near >= 24    # every trial did put at least one quotient into the window where the estimate cannot decide


@pytest.mark.parametrize("T", [5, 300])
def test_two_layer_chain_of_predictors(oracle, T):
    """Fig. 2: the predictors share the network's input, each runs its own cluster of orders layer after
    layer on its own integer activations, and their outputs are added after the last layer only."""
    rng = np.random.default_rng(17 + T)
    I1, O1, O2, bits, K, g, M = 384, 256, 136, 4, 4, 8, 2
    W1, W2 = _w(rng, O1, I1), _w(rng, O2, O1)
    b1 = (rng.standard_normal(O1) * 0.1).astype(np.float32)
    b2 = (rng.standard_normal(O2) * 0.1).astype(np.float32)
    nk1, nk2 = 16, 9
    e1, e2 = oracle.expand(W1, bits, K, g, nk1), oracle.expand(W2, bits, K, g, nk2)
    L1 = H.gpu_expand(H.desc_of(O1, I1, bits, K, g, nk1, M), W1)
    L2 = H.gpu_expand(H.desc_of(O2, O1, bits, K, g, nk2, M), W2)
    split1 = [L1.layout.branch_orders[m] for m in range(M)]
    split2 = [L2.layout.branch_orders[m] for m in range(M)]
    x = rng.standard_normal((T, I1)).astype(np.float32)
    xq, sx = H.gpu_quantize(x)
    xq_o, sx_o = oracle.quantize_act(x)

    # oracle chain
    hq_o, steps = [], []
    k0 = 0
    for m in range(M):
        b = b1 if m == 0 else None
        y = oracle.forward(e1, xq_o, sx_o, k0, k0 + split1[m], bias=b).y
        s = float(np.float32(np.abs(np.maximum(y, 0)).max() / 127))
        steps.append(s)
        hq_o.append(oracle.forward_requantized(e1, xq_o, sx_o, s, k0, k0 + split1[m], bias=b))
        k0 += split1[m]
    y_o, _ = oracle.ensemble(e2, np.stack(hq_o), steps, split2, bias=b2, sum_branches=True)

    # the same chain on the device: no float tensor exists between the layers
    hq, _ = H.gpu_ensemble_q8(L1, [xq] * M, [sx] * M, steps, b1, relu=True)
    for m in range(M):
        np.testing.assert_array_equal(hq[m], hq_o[m])
    hq_d = [torch.from_numpy(h).cuda() for h in hq]
    s_d = [torch.tensor([s], dtype=torch.float32, device="cuda") for s in steps]
    ys, _ = H.gpu_ensemble(L2, hq_d, s_d, b2, sum_branches=True)
    np.testing.assert_array_equal(ys[0].view(np.uint32), y_o.view(np.uint32))


def test_inner_layer_argument_errors(oracle):
    rng = np.random.default_rng(2)
    O, I, T = 64, 128, 40
    W = _w(rng, O, I)
    layer = H.gpu_expand(H.desc_of(O, I, 4, 2, 8, 4, 1), W)
    xq, sx = H.gpu_quantize(rng.standard_normal((T, I)).astype(np.float32))
    # a zero step: every code is zero
    got, _ = H.gpu_ensemble_q8(layer, [xq], [sx], [0.0])
    assert B.pipe_poll_status() == B.PIPE_OK and not got[0].any()
    # a negative step is an argument error reported through the device status
    for kernel in (B.KERNEL_REFERENCE, B.KERNEL_TCGEN05):
        H.gpu_ensemble_q8(layer, [xq], [sx], [-1.0], kernel=kernel)
        assert B.pipe_poll_status() == B.PIPE_ERR_INVALID_ARG
    # the SM-pair kernel on a single token tile (its second CTA then stages zeros): the same codes as the others
    want, _ = H.gpu_ensemble_q8(layer, [xq], [sx], [1.0], kernel=B.KERNEL_REFERENCE)
    got, _ = H.gpu_ensemble_q8(layer, [xq], [sx], [1.0], kernel=B.KERNEL_TCGEN05_PAIR)
    assert B.pipe_poll_status() == B.PIPE_OK and np.array_equal(got[0], want[0])
    # zero tokens: nothing to do
    empty = torch.empty((0, I), dtype=torch.int8, device="cuda")
    got, _ = H.gpu_ensemble_q8(layer, [empty], [sx], [1.0])
    assert got[0].shape == (0, O)


CONV_INNER_CASES = [
    # N, H,  W,  C,   O,  kh, kw, bits, K, g, n_keep, stride, relu
    (2, 16, 16, 128, 128, 3, 3, 4, 3, 8, 6, 1, True),
    (1, 15, 9, 128, 72, 3, 3, 2, 4, 8, 3, 1, True),     # edge patches hang over the output
    (2, 28, 28, 128, 256, 3, 3, 4, 2, 8, 16, 2, False),  # stride 2
    (3, 8, 8, 256, 128, 1, 1, 8, 2, 8, 8, 1, True),
]


@pytest.mark.parametrize("N,Hh,Ww,Cc,O,kh,kw,bits,K,g,n_keep,stride,relu", CONV_INNER_CASES)
def test_requantized_convolution_matches_oracle(oracle, N, Hh, Ww, Cc, O, kh, kw, bits, K, g, n_keep, stride, relu):
    """pipe_expanded_conv2d_q8 on the NHWC tensor == the oracle's inner layer on explicitly lowered im2col rows;
    with O = 128 the int8 output is then fed, as it stands, to a second convolution."""
    rng = np.random.default_rng(N * 1000 + Hh * 10 + Cc + O)
    I = kh * kw * Cc
    W = _w(rng, O, I, heavy=(bits == 2))
    bias = (rng.standard_normal(O) * 0.1).astype(np.float32)
    x4 = np.maximum(rng.standard_normal((N, Hh, Ww, Cc)), 0).astype(np.float32)
    e = oracle.expand(W, bits, K, g, n_keep)
    layer = H.gpu_expand(H.desc_of(O, I, bits, K, g, n_keep), W)
    xq4, sx = H.gpu_quantize(x4.reshape(-1, Cc))
    xq_o, sx_o = oracle.quantize_act(x4.reshape(-1, Cc))

    def lower(xq, n, h, w, c, kh, kw, stride):
        ph, pw = (kh - 1) // 2, (kw - 1) // 2
        ho, wo = (h + 2 * ph - kh) // stride + 1, (w + 2 * pw - kw) // stride + 1
        xp = np.zeros((n, h + 2 * ph, w + 2 * pw, c), np.int8)
        xp[:, ph:ph + h, pw:pw + w] = xq.reshape(n, h, w, c)
        rows = np.zeros((n, ho, wo, kh * kw * c), np.int8)
        for dh in range(kh):
            for dw in range(kw):
                tap = dh * kw + dw
                rows[..., tap * c:(tap + 1) * c] = xp[:, dh:dh + stride * (ho - 1) + 1:stride, dw:dw + stride * (wo - 1) + 1:stride]
        return rows.reshape(-1, kh * kw * c), ho, wo, ph, pw

    rows, Ho, Wo, ph, pw = lower(xq_o, N, Hh, Ww, Cc, kh, kw, stride)
    f = oracle.forward(e, rows, sx_o, bias=bias)
    a = np.maximum(f.y, 0) if relu else f.y
    s_out = float(np.float32(np.quantile(np.abs(a), 0.98) / 127))
    want = oracle.forward_requantized(e, rows, sx_o, s_out, bias=bias, relu=relu)

    def geom_of(n, h, w, c, kh, kw, ph, pw, stride):
        geom = B.ConvGeom()
        geom.batch, geom.height, geom.width, geom.channels = n, h, w, c
        geom.kernel_h, geom.kernel_w, geom.pad_h, geom.pad_w = kh, kw, ph, pw
        geom.stride_h = geom.stride_w = stride
        return geom

    T = N * Ho * Wo
    yq = torch.full((T, O), 99, dtype=torch.int8, device="cuda")
    so = torch.tensor([s_out], dtype=torch.float32, device="cuda")
    part = torch.zeros((T, layer.layout.total_rows), dtype=torch.int32, device="cuda")
    B.pipe_expanded_conv2d_q8(layer.desc, geom_of(N, Hh, Ww, Cc, kh, kw, ph, pw, stride), layer.blob, xq4.view(N, Hh, Ww, Cc),
                              sx, so, yq, torch.from_numpy(bias).cuda(), relu, part)
    torch.cuda.synchronize()
    assert B.pipe_poll_status() == B.PIPE_OK
    np.testing.assert_array_equal(part.cpu().numpy(), f.partials)
    np.testing.assert_array_equal(yq.cpu().numpy(), want)

    if O % 128 == 0:
        # the next convolution reads the int8 NHWC tensor the first one wrote
        O2 = 64
        W2 = _w(rng, O2, 9 * O)
        e2 = oracle.expand(W2, 4, 2, 8, 4)
        layer2 = H.gpu_expand(H.desc_of(O2, 9 * O, 4, 2, 8, 4), W2)
        rows2, Ho2, Wo2, ph2, pw2 = lower(want, N, Ho, Wo, O, 3, 3, 1)
        f2 = oracle.forward(e2, rows2, np.float32(s_out))
        y2 = torch.full((N * Ho2 * Wo2, O2), float("nan"), dtype=torch.float32, device="cuda")
        B.pipe_expanded_conv2d(layer2.desc, geom_of(N, Ho, Wo, O, 3, 3, ph2, pw2, 1), layer2.blob, yq.view(N, Ho, Wo, O), so, y2)
        torch.cuda.synchronize()
        assert B.pipe_poll_status() == B.PIPE_OK
        np.testing.assert_array_equal(y2.cpu().numpy().view(np.uint32), f2.y.view(np.uint32))
