"""GPU-vs-oracle parity on oracle-sized cases: every stage, element by element.
Integer stages (codes, scales, kept lists, int32 partial sums, activation codes) must be bit-exact;
fp32 outputs within 1e-5 relative of the binary64 sum (and, as a stretch, bit-equal to the oracle)."""
import numpy as np
import pytest
import torch

from paper_2311_15806_b200 import binding as B
from paper_2311_15806_b200 import synth
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


# shapes span several tiles and ragged tails in every dimension; g in {1, 4, 8, 16}
EXPAND_CASES = [
    # O,   I,   bits, K, g,  n_keep
    (256, 256, 8, 2, 8, 32),
    (96, 200, 4, 3, 8, 3),
    (80, 1000, 4, 4, 16, 2),
    (64, 328, 2, 5, 4, 5),
    (48, 130, 8, 3, 1, 7),
    (304, 4112, 4, 3, 8, 19),
    (40, 36, 2, 8, 8, 2),
    (8, 8, 4, 2, 8, 1),
]


@pytest.mark.parametrize("O,I,bits,K,g,n_keep", EXPAND_CASES)
def test_expand_weights_bit_exact(oracle, O, I, bits, K, g, n_keep):
    rng = np.random.default_rng(O * 31 + I)
    W = _w(rng, O, I, heavy=True)
    W[O // 2] = 0.0                      # an all-zero row
    W[1] = W[0]                          # equal rows
    e = oracle.expand(W, bits, K, g, n_keep)
    layer = H.gpu_expand(H.desc_of(O, I, bits, K, g, n_keep), W)
    H.assert_expansion_matches(layer, e, oracle)


@pytest.mark.parametrize("bits", [8, 4, 2])
def test_expand_weights_at_rounding_boundaries(oracle, bits):
    """Rows whose entries sit on, and a few ulps beside, the boundaries (k + 1/2) * s of their own scale: the
    codes are defined by the IEEE quotient, whatever shortcut the kernel takes elsewhere (Eq. 1)."""
    qmax = (1 << (bits - 1)) - 1
    rows = []
    for amax in (1.0, 0.0372, 3e-5, 911.0):
        s = np.float32(np.float32(amax) / np.float32(qmax))
        ks = np.arange(-qmax, qmax, dtype=np.float64) + 0.5
        base = (ks * np.float64(s)).astype(np.float32)
        for shift in range(-3, 4):
            v = base.copy()
            for _ in range(abs(shift)):
                v = np.nextafter(v, np.float32(np.inf if shift > 0 else -np.inf), dtype=np.float32)
            row = np.zeros(256, np.float32)
            reps = -(-255 // len(v))
            row[:255] = np.tile(v, reps)[:255]
            row[255] = np.float32(amax)            # pins the row's absmax
            rows.append(row)
    W = np.stack(rows).astype(np.float32)
    W = np.concatenate([W, np.zeros((32 - len(W) % 32 if len(W) % 32 else 0, 256), np.float32)])
    O = W.shape[0]
    e = oracle.expand(W, bits, 3, 8, O // 8)
    layer = H.gpu_expand(H.desc_of(O, 256, bits, 3, 8, O // 8), W)
    H.assert_expansion_matches(layer, e, oracle)


def test_expand_weights_strided_and_tied_groups(oracle):
    rng = np.random.default_rng(5)
    O, I, g = 64, 72, 8
    big = rng.standard_normal((O, I + 9)).astype(np.float32)
    # tie the scores of several groups: copy group 1 into groups 3 and 6
    big[3 * g:4 * g] = big[g:2 * g]
    big[6 * g:7 * g] = big[g:2 * g]
    Wd = torch.from_numpy(big).cuda()[:, 3:3 + I]            # pitch I+9, misaligned rows
    W = np.ascontiguousarray(big[:, 3:3 + I])
    d = H.desc_of(O, I, 4, 3, g, 2)
    layer = B.expand(d, Wd)
    torch.cuda.synchronize()
    H.assert_expansion_matches(layer, oracle.expand(W, 4, 3, g, 2), oracle)


def test_expand_weights_is_deterministic(oracle):
    rng = np.random.default_rng(6)
    W = _w(rng, 128, 512)
    d = H.desc_of(128, 512, 4, 4, 8, 8)
    blobs = [H.gpu_expand(d, W).blob.cpu().numpy() for _ in range(3)]
    lay = B.pipe_layout(d)
    for k in range(4):
        for off, n in [(lay.codes_off[k], lay.rows[k] * lay.canon_row_bytes), (lay.scales_off[k], lay.rows[k] * 4),
                       (lay.kcodes_off[k], lay.rows[k] * lay.kernel_row_bytes)]:
            assert (blobs[0][off:off + n] == blobs[1][off:off + n]).all()
            assert (blobs[0][off:off + n] == blobs[2][off:off + n]).all()


def test_nonfinite_weights_raise_device_status():
    W = np.ones((16, 32), np.float32)
    W[3, 5] = np.nan
    d = H.desc_of(16, 32, 4, 2, 8, 1)
    B.expand(d, torch.from_numpy(W).cuda())
    assert B.pipe_poll_status() == B.PIPE_ERR_NONFINITE
    assert B.pipe_poll_status() == B.PIPE_OK   # cleared by the poll


@pytest.mark.parametrize("T,I", [(64, 256), (1, 4096), (7, 33), (130, 1000), (300, 2304), (0, 64)])
def test_quantize_act_bit_exact(oracle, T, I):
    rng = np.random.default_rng(T * 7 + I)
    x = (rng.standard_normal((T, I)) * 2.5).astype(np.float32)
    if T > 2:
        x[:, ::37] *= 20
    xq, sx = H.gpu_quantize(x)
    if T == 0:
        assert float(sx.cpu()) == 0.0
        return
    xq_o, sx_o = oracle.quantize_act(x)
    assert sx.cpu().numpy().view(np.uint32)[0] == np.float32(sx_o).view(np.uint32)
    np.testing.assert_array_equal(xq.cpu().numpy(), xq_o)


def test_quantize_act_at_rounding_boundaries(oracle):
    """Values placed on, and one or two ulps beside, the rounding boundaries (k + 1/2) * lambda_x: the code is
    defined by the IEEE quotient, so a kernel that estimates the quotient must fall back to the true
    division there (Eq. 1 with the division reading)."""
    rng = np.random.default_rng(5)
    for amax in (127.0, 3.1415927, 1e-3, 77.7):
        s = np.float32(np.float32(amax) / np.float32(127.0))
        ks = np.arange(-127, 127, dtype=np.float64) + 0.5
        base = (ks * np.float64(s)).astype(np.float32)
        cols = [base]
        v = base.copy()
        for _ in range(3):
            v = np.nextafter(v, np.float32(np.inf), dtype=np.float32)
            cols.append(v.copy())
        v = base.copy()
        for _ in range(3):
            v = np.nextafter(v, np.float32(-np.inf), dtype=np.float32)
            cols.append(v.copy())
        x = np.stack(cols).astype(np.float32)                     # [7, 254]
        x = np.concatenate([x, (rng.standard_normal((5, 254)) * amax / 3).astype(np.float32).clip(-amax, amax)])
        x = np.concatenate([x, np.zeros((12, 2), np.float32)], axis=1)   # 256 columns: the contiguous fast path
        x[0, -1] = np.float32(amax)                                # pins the tensor's absmax
        xq, sx = H.gpu_quantize(x)
        xq_o, sx_o = oracle.quantize_act(x)
        assert sx.cpu().numpy().view(np.uint32)[0] == np.float32(sx_o).view(np.uint32)
        np.testing.assert_array_equal(xq.cpu().numpy(), xq_o)
        # the same through a static scale that is not absmax / 127 (clamping and large quotients)
        xq, _ = H.gpu_quantize(x, static_scale=float(s) / 3)
        xq_o, _ = oracle.quantize_act(x, static_scale=float(s) / 3)
        np.testing.assert_array_equal(xq.cpu().numpy(), xq_o)


def test_quantize_act_static_scale_zero_and_strided(oracle):
    rng = np.random.default_rng(11)
    x = (rng.standard_normal((9, 50)) * 100).astype(np.float32)
    xq, sx = H.gpu_quantize(x, static_scale=0.5)
    xq_o, _ = oracle.quantize_act(x, static_scale=0.5)
    np.testing.assert_array_equal(xq.cpu().numpy(), xq_o)
    xq, sx = H.gpu_quantize(np.zeros((5, 20), np.float32))
    assert float(sx.cpu()) == 0.0 and not xq.cpu().numpy().any()
    big = torch.from_numpy(rng.standard_normal((12, 77)).astype(np.float32)).cuda()
    view = big[:, 5:5 + 64]
    xq, sx = H.gpu_quantize(None, xd=view)
    xq_o, sx_o = oracle.quantize_act(view.cpu().numpy())
    np.testing.assert_array_equal(xq.cpu().numpy(), xq_o)
    bad = np.ones((4, 16), np.float32)
    bad[2, 3] = np.inf
    H.gpu_quantize(bad)
    assert B.pipe_poll_status() == B.PIPE_ERR_NONFINITE


FORWARD_CASES = [
    # O,   I,    T,  bits, K, g, n_keep, M
    (256, 256, 64, 8, 2, 8, 32, 1),
    (96, 200, 70, 4, 3, 8, 3, 1),
    (192, 1000, 150, 4, 4, 8, 12, 2),
    (128, 328, 33, 2, 8, 16, 2, 4),
    (48, 130, 5, 8, 3, 1, 7, 3),
    (304, 2304, 131, 4, 3, 8, 19, 1),
    (264, 512, 1, 4, 4, 8, 17, 2),
    (264, 512, 16, 4, 4, 8, 17, 2),
    (128, 128, 128, 8, 1, 8, 16, 1),
    (264, 1008, 700, 4, 4, 8, 17, 2),
    (512, 272, 1000, 2, 8, 16, 8, 4),
    (200, 144, 260, 8, 3, 8, 5, 3),
    (640, 640, 129, 4, 6, 32, 3, 1),
    (128, 328, 7, 2, 8, 16, 2, 4),
    (256, 256, 9, 8, 2, 8, 32, 1),
    (304, 2304, 16, 4, 3, 8, 19, 1),
    (72, 4112, 3, 4, 5, 8, 4, 2),
    (136, 1000, 12, 2, 4, 8, 9, 1),
    # decode kernel: int8 codes; eight orders in one branch (four order pairs per slab); ternary with an odd
    # number of reduction blocks; more slabs per CTA than one pass holds
    (256, 384, 9, 8, 2, 8, 16, 1),
    (320, 1024, 7, 2, 8, 8, 10, 1),
    (200, 1152, 16, 2, 3, 8, 11, 1),
    (24832, 128, 5, 4, 2, 8, 1552, 1),
    # 18 slabs per CTA on 148 SMs: nearly every slab slot of a consumer warp is taken (the kernel without per-slab branches)
    (21312, 128, 3, 4, 2, 8, 1000, 1),
    (21312, 256, 8, 2, 2, 16, 700, 1),
    # ... and with 6, 10 and 14 slabs per CTA (two, three, four slab slots per warp), up to 8 and up to 16 tokens
    (7104, 128, 12, 4, 2, 8, 400, 1),
    (7104, 256, 2, 8, 2, 8, 300, 1),
    (11840, 128, 16, 4, 2, 8, 700, 1),
    (16576, 128, 1, 2, 2, 16, 500, 1),
]


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("O,I,T,bits,K,g,n_keep,M", FORWARD_CASES)
def test_forward_matches_oracle(oracle, kernel, O, I, T, bits, K, g, n_keep, M, int8_copy=False):
    rng = np.random.default_rng(O + 3 * I + 5 * T)
    W = _w(rng, O, I, heavy=(bits == 2))
    bias = rng.standard_normal(O).astype(np.float32)
    e = oracle.expand(W, bits, K, g, n_keep)
    d = H.desc_of(O, I, bits, K, g, n_keep, M, int8_copy=int8_copy)
    layer = H.gpu_expand(d, W)
    H.assert_expansion_matches(layer, e, oracle, check_kernel_layout=False)
    split = [layer.layout.branch_orders[m] for m in range(M)]
    xs = [(rng.standard_normal((T, I)) * (1 + m)).astype(np.float32) for m in range(M)]
    q = [H.gpu_quantize(x) for x in xs]
    qo = [oracle.quantize_act(x) for x in xs]
    for (xq, sx), (xq_o, sx_o) in zip(q, qo):
        np.testing.assert_array_equal(xq.cpu().numpy(), xq_o)

    # (1) the whole expanded layer on one input
    try:
        y, part = H.gpu_linear(layer, q[0][0], q[0][1], bias, kernel=kernel)
    except B.PipeError as ex:
        if ex.status == B.PIPE_ERR_UNSUPPORTED and kernel != B.KERNEL_AUTO:
            pytest.skip("this kernel does not take this shape (the automatic choice falls back)")
        raise
    f = oracle.forward(e, qo[0][0], qo[0][1], bias=bias)
    np.testing.assert_array_equal(part, f.partials)
    H.assert_outputs_close(y, f, "expanded_linear")
    np.testing.assert_array_equal(y.view(np.uint32), f.y.view(np.uint32))   # same operation order => same bits

    # (2) grouped ensemble, distinct inputs, per-branch outputs
    ys, part = H.gpu_ensemble(layer, [a for a, _ in q], [b for _, b in q], bias, kernel=kernel)
    k0 = 0
    want_part = np.zeros_like(part)
    for m in range(M):
        fm = oracle.forward(e, qo[m][0], qo[m][1], k0, k0 + split[m], bias=bias if m == 0 else None)
        H.assert_outputs_close(ys[m], fm, f"branch {m}")
        np.testing.assert_array_equal(ys[m].view(np.uint32), fm.y.view(np.uint32))
        lo, hi = e.row_off(k0), e.row_off(k0 + split[m])
        want_part[:, lo:hi] = fm.partials[:, lo:hi]
        k0 += split[m]
    np.testing.assert_array_equal(part, want_part)

    # (3) shared input, summed after the layer: partials equal those of the un-split layer
    ys, part = H.gpu_ensemble(layer, [q[0][0]] * M, [q[0][1]] * M, bias, sum_branches=True, kernel=kernel)
    np.testing.assert_array_equal(part, f.partials)
    y_o, _ = oracle.ensemble(e, np.stack([qo[0][0]] * M), [qo[0][1]] * M, split, bias=bias, sum_branches=True)
    np.testing.assert_array_equal(ys[0].view(np.uint32), y_o.view(np.uint32))
    assert (np.abs(ys[0] - f.y64) <= H.REL_TOL * f.yabs + 1e-30).all()


@pytest.mark.parametrize("kernel", [B.KERNEL_AUTO, B.KERNEL_TCGEN05_PAIR, B.KERNEL_TCGEN05, B.KERNEL_STREAM])
@pytest.mark.parametrize("O,I,T,bits,K,g,n_keep,M", [c for c in FORWARD_CASES if c[5] % 8 == 0])
def test_forward_with_int8_copy_matches_oracle(oracle, kernel, O, I, T, bits, K, g, n_keep, M):
    """A layer that also keeps its codes as int8 in the tensor-core operand layout: the copy is what the definition
    says, the kernels that use it (the SM-pair kernel) and those that do not give the oracle's bits."""
    test_forward_matches_oracle(oracle, kernel, O, I, T, bits, K, g, n_keep, M, int8_copy=True)


@pytest.mark.parametrize("kernel,T", [(B.KERNEL_TCGEN05_PAIR, 300), (B.KERNEL_STREAM, 7), (B.KERNEL_STREAM, 16), (B.KERNEL_AUTO, 1)])
def test_summed_ensemble_on_a_shared_input_is_one_launch(oracle, kernel, T):
    """Predictors that share their input and are summed after the layer (Sec. 3.2) run as ONE launch of the SM-pair
    kernel (of the weight-streaming kernel for up to 16 tokens) on the cluster of all orders; with distinct inputs it is
    one launch per predictor.  Both give the oracle's bits (each predictor's chain from zero, the bias closing the
    first, the chains added in ascending order)."""
    O, I, bits, K, g, n_keep, M = 512, 640, 4, 6, 8, 24, 3
    rng = np.random.default_rng(77)
    W = _w(rng, O, I)
    bias = rng.standard_normal(O).astype(np.float32)
    e = oracle.expand(W, bits, K, g, n_keep)
    layer = H.gpu_expand(H.desc_of(O, I, bits, K, g, n_keep, M), W)
    split = [layer.layout.branch_orders[m] for m in range(M)]
    xs = [(rng.standard_normal((T, I)) * (1 + m)).astype(np.float32) for m in range(M)]
    q = [H.gpu_quantize(x) for x in xs]
    qo = [oracle.quantize_act(x) for x in xs]
    bd = torch.from_numpy(bias).cuda()
    for shared in (True, False):
        xq = [q[0][0]] * M if shared else [a for a, _ in q]
        sx = [q[0][1]] * M if shared else [b for _, b in q]
        y = torch.full((T, O), float("nan"), dtype=torch.float32, device="cuda")
        B.pipe_diag_select_kernel(kernel)
        try:
            before = B.pipe_launch_count()
            B.pipe_ensemble_forward(layer.desc, layer.blob, xq, sx, [y], bd, True, None)
            launches = B.pipe_launch_count() - before
            torch.cuda.synchronize()
        finally:
            B.pipe_diag_select_kernel(B.KERNEL_AUTO)
        assert B.pipe_poll_status() == B.PIPE_OK
        assert launches == (1 if shared else M)
        xo = np.stack([qo[0][0]] * M) if shared else np.stack([a for a, _ in qo])
        so = [qo[0][1]] * M if shared else [b for _, b in qo]
        y_o, _ = oracle.ensemble(e, xo, so, split, bias=bias, sum_branches=True)
        np.testing.assert_array_equal(y.cpu().numpy().view(np.uint32), y_o.view(np.uint32))


def test_forward_zero_tokens_and_strided_io(oracle):
    rng = np.random.default_rng(77)
    O, I, T = 64, 96, 10
    W = _w(rng, O, I)
    e = oracle.expand(W, 4, 2, 8, 4)
    layer = H.gpu_expand(H.desc_of(O, I, 4, 2, 8, 4), W)
    x = rng.standard_normal((T, I)).astype(np.float32)
    xq_o, sx_o = oracle.quantize_act(x)
    xq_big = torch.zeros((T, I + 32), dtype=torch.int8, device="cuda")
    xq_big[:, 16:16 + I] = torch.from_numpy(xq_o).cuda()
    y_big = torch.zeros((T, O + 8), dtype=torch.float32, device="cuda")
    sx = torch.tensor([sx_o], dtype=torch.float32, device="cuda")
    B.pipe_expanded_linear(layer.desc, layer.blob, xq_big[:, 16:16 + I], sx, y_big[:, 4:4 + O])
    torch.cuda.synchronize()
    f = oracle.forward(e, xq_o, sx_o)
    np.testing.assert_array_equal(y_big[:, 4:4 + O].cpu().numpy().view(np.uint32), f.y.view(np.uint32))
    assert not y_big[:, :4].any() and not y_big[:, 4 + O:].any()
    empty = torch.empty((0, I), dtype=torch.int8, device="cuda")
    B.pipe_expanded_linear(layer.desc, layer.blob, empty, sx, torch.empty((0, O), dtype=torch.float32, device="cuda"))
    assert B.pipe_poll_status() == B.PIPE_OK


CONV_CASES = [
    # N, H,  W,  C,   O,  kh, kw, bits, K, g, n_keep, stride, pad (None: (k - 1) / 2)
    (2, 16, 8, 128, 64, 3, 3, 4, 3, 8, 2, 1, None),
    (1, 8, 24, 128, 72, 3, 3, 8, 2, 8, 3, 1, None),      # odd number of 8x8 patches: the last tile is half empty
    (3, 8, 8, 256, 136, 1, 1, 2, 4, 8, 5, 1, None),      # 1x1: no halo
    (1, 24, 16, 128, 40, 5, 3, 4, 2, 8, 5, 1, None),     # rectangular filter, two rows/columns of padding
    (2, 14, 14, 128, 64, 3, 3, 4, 3, 8, 2, 1, None),     # output not a multiple of the 8x8 patch: edge patches hang over
    (1, 15, 9, 128, 40, 3, 3, 4, 2, 8, 5, 2, None),      # stride 2, odd sizes: 8 x 5 outputs
    (2, 16, 16, 256, 72, 1, 1, 8, 2, 8, 3, 2, None),     # strided 1x1 (a downsampling shortcut)
    (1, 28, 28, 128, 64, 3, 3, 4, 3, 8, 2, 2, None),     # 28 -> 14
    (1, 12, 20, 128, 48, 3, 3, 2, 3, 8, 2, 1, (0, 0)),   # no padding: 10 x 18 outputs
]


@pytest.mark.parametrize("kernel", [B.KERNEL_AUTO, B.KERNEL_TCGEN05_PAIR])
@pytest.mark.parametrize("N,Hh,Ww,Cc,O,kh,kw,bits,K,g,n_keep,stride,pad", CONV_CASES)
def test_implicit_convolution_matches_oracle(oracle, kernel, N, Hh, Ww, Cc, O, kh, kw, bits, K, g, n_keep, stride, pad):
    """pipe_expanded_conv2d on the NHWC tensor == the oracle on explicitly lowered im2col rows."""
    rng = np.random.default_rng(N * 1000 + Hh * 10 + Cc)
    I = kh * kw * Cc
    W = _w(rng, O, I, heavy=(bits == 2))
    bias = rng.standard_normal(O).astype(np.float32)
    x4 = np.maximum(rng.standard_normal((N, Hh, Ww, Cc)), 0).astype(np.float32)
    e = oracle.expand(W, bits, K, g, n_keep)
    layer = H.gpu_expand(H.desc_of(O, I, bits, K, g, n_keep), W)
    xq4, sx = H.gpu_quantize(x4.reshape(-1, Cc))
    xq_o, sx_o = oracle.quantize_act(x4.reshape(-1, Cc))
    np.testing.assert_array_equal(xq4.cpu().numpy(), xq_o)
    # explicit lowering on the host (pad_h may differ from pad_w: lower by hand)
    ph, pw = ((kh - 1) // 2, (kw - 1) // 2) if pad is None else pad
    Ho, Wo = (Hh + 2 * ph - kh) // stride + 1, (Ww + 2 * pw - kw) // stride + 1
    xp = np.zeros((N, Hh + 2 * ph, Ww + 2 * pw, Cc), np.int8)
    xp[:, ph:ph + Hh, pw:pw + Ww] = xq_o.reshape(N, Hh, Ww, Cc)
    rows = np.zeros((N, Ho, Wo, kh * kw * Cc), np.int8)
    for dh in range(kh):
        for dw in range(kw):
            tap = dh * kw + dw
            rows[..., tap * Cc:(tap + 1) * Cc] = xp[:, dh:dh + stride * (Ho - 1) + 1:stride, dw:dw + stride * (Wo - 1) + 1:stride]
    f = oracle.forward(e, rows.reshape(-1, I), sx_o, bias=bias)
    geom = B.ConvGeom()
    geom.batch, geom.height, geom.width, geom.channels = N, Hh, Ww, Cc
    geom.kernel_h, geom.kernel_w, geom.pad_h, geom.pad_w = kh, kw, ph, pw
    geom.stride_h = geom.stride_w = stride
    T = N * Ho * Wo
    y = torch.full((T, O), float("nan"), dtype=torch.float32, device="cuda")
    part = torch.zeros((T, layer.layout.total_rows), dtype=torch.int32, device="cuda")
    B.pipe_diag_select_kernel(kernel)
    try:
        B.pipe_expanded_conv2d(layer.desc, geom, layer.blob, xq4.view(N, Hh, Ww, Cc), sx, y, torch.from_numpy(bias).cuda(), part)
    except B.PipeError as ex:
        if ex.status == B.PIPE_ERR_UNSUPPORTED and kernel != B.KERNEL_AUTO:
            pytest.skip("the two-SM kernel needs at least two token tiles")
        raise
    finally:
        B.pipe_diag_select_kernel(B.KERNEL_AUTO)
    torch.cuda.synchronize()
    assert B.pipe_poll_status() == B.PIPE_OK
    np.testing.assert_array_equal(part.cpu().numpy(), f.partials)
    H.assert_outputs_close(y.cpu().numpy(), f, "conv2d")
    np.testing.assert_array_equal(y.cpu().numpy().view(np.uint32), f.y.view(np.uint32))


def test_convolution_shapes_outside_the_fast_path_are_refused():
    layer_desc = H.desc_of(64, 9 * 96, 4, 2, 8, 2)
    lay = B.pipe_layout(layer_desc)
    blob = B.alloc_bytes(lay.blob_bytes)
    geom = B.ConvGeom()
    geom.batch, geom.height, geom.width, geom.channels = 1, 8, 8, 96
    geom.kernel_h, geom.kernel_w, geom.pad_h, geom.pad_w = 3, 3, 1, 1
    xq = torch.zeros((1, 8, 8, 96), dtype=torch.int8, device="cuda")
    sx = torch.ones(1, device="cuda")
    y = torch.zeros((64, 64), device="cuda")
    with pytest.raises(B.PipeError) as ei:
        B.pipe_expanded_conv2d(layer_desc, geom, blob, xq, sx, y)
    assert ei.value.status == B.PIPE_ERR_UNSUPPORTED
    geom.pad_h = 3   # as much padding as the filter is high: no output row would see the image
    with pytest.raises(B.PipeError) as ei:
        B.pipe_expanded_conv2d(layer_desc, geom, blob, xq, sx, y)
    assert ei.value.status == B.PIPE_ERR_SHAPE


def test_launch_counter_moves():
    before = B.pipe_launch_count()
    H.gpu_quantize(np.ones((4, 16), np.float32))
    assert B.pipe_launch_count() >= before + 2


def test_forward_is_deterministic_across_repeated_runs(oracle):
    """The same call three times over gives the same bits: integer sums, fp32 outputs, and a re-expansion of the same
    weights (no atomics or race decides anything in the path)."""
    rng = np.random.default_rng(2024)
    O, I, T, bits, K, g, n_keep, M = 256, 640, 700, 4, 4, 8, 16, 2
    W = _w(rng, O, I)
    d = H.desc_of(O, I, bits, K, g, n_keep, M)
    xs = [rng.standard_normal((T, I)).astype(np.float32) for _ in range(M)]
    ref = None
    for rep in range(3):
        layer = H.gpu_expand(d, W)
        q = [H.gpu_quantize(x) for x in xs]
        ys, part = H.gpu_ensemble(layer, [a for a, _ in q], [b for _, b in q], None)
        sections = np.concatenate([t.cpu().numpy().view(np.uint8).reshape(-1) for k in range(K)
                                   for t in (layer.codes(k), layer.kcodes(k), layer.scales(k), layer.kept(k), layer.cum(k))])
        got = (sections, [y.view(np.uint32).copy() for y in ys], part.copy())
        if ref is None:
            ref = got
            continue
        np.testing.assert_array_equal(got[0], ref[0])
        for a, b in zip(got[1], ref[1]):
            np.testing.assert_array_equal(a, b)
        np.testing.assert_array_equal(got[2], ref[2])
    for T_small in (1, 16):      # the small-token path too
        q = [H.gpu_quantize(x[:T_small]) for x in xs]
        outs = [H.gpu_ensemble(layer, [a for a, _ in q], [b for _, b in q], None)[0] for _ in range(3)]
        for o in outs[1:]:
            for a, b in zip(o, outs[0]):
                np.testing.assert_array_equal(a.view(np.uint32), b.view(np.uint32))


def _lower_im2col(xq_nhwc, kh, kw, ph, pw, stride):
    """Explicit lowering of an int8 NHWC tensor to the rows of the convolution's GEMM (reduction index (tap, channel))."""
    N, Hh, Ww, Cc = xq_nhwc.shape
    Ho, Wo = (Hh + 2 * ph - kh) // stride + 1, (Ww + 2 * pw - kw) // stride + 1
    xp = np.zeros((N, Hh + 2 * ph, Ww + 2 * pw, Cc), np.int8)
    xp[:, ph:ph + Hh, pw:pw + Ww] = xq_nhwc
    rows = np.zeros((N, Ho, Wo, kh * kw * Cc), np.int8)
    for dh in range(kh):
        for dw in range(kw):
            tap = dh * kw + dw
            rows[..., tap * Cc:(tap + 1) * Cc] = xp[:, dh:dh + stride * (Ho - 1) + 1:stride, dw:dw + stride * (Wo - 1) + 1:stride]
    return rows.reshape(N * Ho * Wo, kh * kw * Cc), Ho, Wo


ENSEMBLE_CONV_CASES = [
    # N, H,  W,  C,   O,  kh, kw, bits, K, g, n_keep, M, stride, sum
    (2, 16, 16, 128, 64, 3, 3, 4, 4, 8, 4, 2, 1, False),
    (1, 14, 14, 128, 72, 3, 3, 4, 3, 8, 3, 3, 1, False),    # edge patches hang over; three predictors of one order each
    (2, 16, 16, 256, 80, 1, 1, 2, 4, 16, 2, 2, 2, False),   # strided 1x1, ternary
    (1, 15, 17, 128, 64, 3, 3, 4, 4, 8, 4, 2, 2, True),     # summed: one launch per predictor, in order
    (2, 12, 12, 128, 48, 3, 3, 8, 2, 8, 3, 2, 1, True),
    (1, 15, 11, 256, 48, 1, 3, 2, 4, 8, 2, 3, 1, False),    # ternary with groups of 8: the one-SM kernel's turn
    (3, 15, 22, 128, 72, 5, 3, 2, 4, 8, 4, 2, 2, True),
]


@pytest.mark.parametrize("N,Hh,Ww,Cc,O,kh,kw,bits,K,g,n_keep,M,stride,summed", ENSEMBLE_CONV_CASES)
def test_ensemble_convolution_matches_oracle(oracle, N, Hh, Ww, Cc, O, kh, kw, bits, K, g, n_keep, M, stride, summed):
    """pipe_ensemble_conv2d (Sec. 3.2 on a convolution: predictor m applies its cluster of orders to its own NHWC
    input) == the oracle's ensemble on explicitly lowered im2col rows of every predictor's input."""
    rng = np.random.default_rng(N * 1000 + Hh * 10 + Cc + M)
    I = kh * kw * Cc
    W = _w(rng, O, I, heavy=(bits == 2))
    bias = rng.standard_normal(O).astype(np.float32)
    e = oracle.expand(W, bits, K, g, n_keep)
    layer = H.gpu_expand(H.desc_of(O, I, bits, K, g, n_keep, M), W)
    split = oracle.balanced_split(K, M)
    ph, pw = (kh - 1) // 2, (kw - 1) // 2
    xq_gpu, sx_gpu, rows_m, sx_o = [], [], [], []
    for m in range(M):
        x4 = (np.maximum(rng.standard_normal((N, Hh, Ww, Cc)), 0) * (1.0 + m)).astype(np.float32)
        xq4, sx = H.gpu_quantize(x4.reshape(-1, Cc))
        xq_o, s_o = oracle.quantize_act(x4.reshape(-1, Cc))
        np.testing.assert_array_equal(xq4.cpu().numpy(), xq_o)
        rows, Ho, Wo = _lower_im2col(xq_o.reshape(N, Hh, Ww, Cc), kh, kw, ph, pw, stride)
        xq_gpu.append(xq4.view(N, Hh, Ww, Cc))
        sx_gpu.append(sx)
        rows_m.append(rows)
        sx_o.append(s_o)
    want_y, want_part = oracle.ensemble(e, np.stack(rows_m), sx_o, split, bias=bias, sum_branches=summed)
    geom = B.ConvGeom()
    geom.batch, geom.height, geom.width, geom.channels = N, Hh, Ww, Cc
    geom.kernel_h, geom.kernel_w, geom.pad_h, geom.pad_w = kh, kw, ph, pw
    geom.stride_h = geom.stride_w = stride
    T = N * Ho * Wo
    ys = [torch.full((T, O), float("nan"), dtype=torch.float32, device="cuda") for _ in range(1 if summed else M)]
    part = torch.zeros((T, layer.layout.total_rows), dtype=torch.int32, device="cuda")
    B.pipe_ensemble_conv2d(layer.desc, geom, layer.blob, xq_gpu, sx_gpu, ys, torch.from_numpy(bias).cuda(), summed, part)
    torch.cuda.synchronize()
    assert B.pipe_poll_status() == B.PIPE_OK
    np.testing.assert_array_equal(part.cpu().numpy(), want_part)
    got = ys[0].cpu().numpy() if summed else np.stack([y.cpu().numpy() for y in ys])
    np.testing.assert_array_equal(got.view(np.uint32), want_y.view(np.uint32))


@pytest.mark.parametrize("N,Hh,Ww,Cc,O,kh,kw,bits,K,g,n_keep,M,stride", [
    (1, 15, 17, 128, 64, 3, 3, 4, 4, 8, 4, 2, 2), (2, 12, 12, 128, 48, 3, 3, 8, 3, 8, 3, 3, 1), (1, 16, 16, 256, 96, 1, 1, 2, 6, 16, 3, 3, 1)])
def test_summed_ensemble_convolution_on_a_shared_input(oracle, N, Hh, Ww, Cc, O, kh, kw, bits, K, g, n_keep, M, stride):
    """The predictors of a first convolution share the image and are summed after the layer: one launch on the cluster of
    all orders (the chains closed and added in registers), the oracle's bits."""
    rng = np.random.default_rng(N * 977 + Hh * 13 + Cc + M)
    I = kh * kw * Cc
    W = _w(rng, O, I, heavy=(bits == 2))
    bias = rng.standard_normal(O).astype(np.float32)
    e = oracle.expand(W, bits, K, g, n_keep)
    layer = H.gpu_expand(H.desc_of(O, I, bits, K, g, n_keep, M), W)
    split = oracle.balanced_split(K, M)
    ph, pw = (kh - 1) // 2, (kw - 1) // 2
    x4 = np.maximum(rng.standard_normal((N, Hh, Ww, Cc)), 0).astype(np.float32)
    xq4, sx = H.gpu_quantize(x4.reshape(-1, Cc))
    xq_o, s_o = oracle.quantize_act(x4.reshape(-1, Cc))
    rows, Ho, Wo = _lower_im2col(xq_o.reshape(N, Hh, Ww, Cc), kh, kw, ph, pw, stride)
    want_y, want_part = oracle.ensemble(e, np.stack([rows] * M), [s_o] * M, split, bias=bias, sum_branches=True)
    geom = B.ConvGeom()
    geom.batch, geom.height, geom.width, geom.channels = N, Hh, Ww, Cc
    geom.kernel_h, geom.kernel_w, geom.pad_h, geom.pad_w = kh, kw, ph, pw
    geom.stride_h = geom.stride_w = stride
    T = N * Ho * Wo
    y = torch.full((T, O), float("nan"), dtype=torch.float32, device="cuda")
    part = torch.zeros((T, layer.layout.total_rows), dtype=torch.int32, device="cuda")
    B.pipe_diag_select_kernel(B.KERNEL_TCGEN05_PAIR)   # (the automatic choice sends layers this small to the one-SM kernel)
    try:
        before = B.pipe_launch_count()
        B.pipe_ensemble_conv2d(layer.desc, geom, layer.blob, [xq4.view(N, Hh, Ww, Cc)] * M, [sx] * M, [y], torch.from_numpy(bias).cuda(), True, part)
        launches = B.pipe_launch_count() - before
        torch.cuda.synchronize()
    finally:
        B.pipe_diag_select_kernel(B.KERNEL_AUTO)
    assert B.pipe_poll_status() == B.PIPE_OK
    assert launches == 1
    np.testing.assert_array_equal(part.cpu().numpy(), want_part)
    np.testing.assert_array_equal(y.cpu().numpy().view(np.uint32), want_y.view(np.uint32))


def test_ensemble_convolution_inner_layer_matches_oracle(oracle):
    """pipe_ensemble_conv2d_q8: every predictor's int8 output equals forward -> ReLU -> quantize(static step) of the
    oracle on the lowered rows of that predictor's input."""
    rng = np.random.default_rng(77)
    N, Hh, Ww, Cc, O, kh, kw, bits, K, g, n_keep, M = 2, 16, 16, 128, 64, 3, 3, 4, 4, 8, 4, 2
    I = kh * kw * Cc
    W = _w(rng, O, I)
    bias = rng.standard_normal(O).astype(np.float32)
    e = oracle.expand(W, bits, K, g, n_keep)
    layer = H.gpu_expand(H.desc_of(O, I, bits, K, g, n_keep, M), W)
    split = oracle.balanced_split(K, M)
    begin = np.concatenate([[0], np.cumsum(split)]).astype(int)
    steps = [0.05, 0.11]
    xq_gpu, sx_gpu, want = [], [], []
    for m in range(M):
        x4 = np.maximum(rng.standard_normal((N, Hh, Ww, Cc)), 0).astype(np.float32)
        xq4, sx = H.gpu_quantize(x4.reshape(-1, Cc))
        xq_o, s_o = oracle.quantize_act(x4.reshape(-1, Cc))
        rows, Ho, Wo = _lower_im2col(xq_o.reshape(N, Hh, Ww, Cc), kh, kw, 1, 1, 1)
        xq_gpu.append(xq4.view(N, Hh, Ww, Cc))
        sx_gpu.append(sx)
        want.append(oracle.forward_requantized(e, rows, s_o, steps[m], int(begin[m]), int(begin[m + 1]),
                                               bias=bias if m == 0 else None, relu=True))
    geom = B.ConvGeom()
    geom.batch, geom.height, geom.width, geom.channels = N, Hh, Ww, Cc
    geom.kernel_h, geom.kernel_w, geom.pad_h, geom.pad_w = kh, kw, 1, 1
    geom.stride_h = geom.stride_w = 1
    T = N * Ho * Wo
    yq = [torch.full((T, O), 99, dtype=torch.int8, device="cuda") for _ in range(M)]
    so = [torch.tensor([s], dtype=torch.float32, device="cuda") for s in steps]
    B.pipe_ensemble_conv2d_q8(layer.desc, geom, layer.blob, xq_gpu, sx_gpu, so, yq, torch.from_numpy(bias).cuda(), True)
    torch.cuda.synchronize()
    assert B.pipe_poll_status() == B.PIPE_OK
    for m in range(M):
        np.testing.assert_array_equal(yq[m].cpu().numpy(), want[m])


LOWER_CASES = [
    # N, H, W, C, kh, kw, pad, stride, pitch_extra
    (2, 20, 18, 3, 7, 7, 3, 2, 13),      # a first layer: 7 x 7 on three channels, stride 2 (I = 147, pitch 160)
    (1, 9, 11, 24, 3, 3, 1, 1, 0),       # channels not a multiple of 16
    (2, 8, 8, 64, 3, 3, 1, 1, 0),        # 16-byte pieces
    (1, 10, 6, 96, 1, 1, 0, 2, 32),
]


@pytest.mark.parametrize("N,Hh,Ww,Cc,kh,kw,pad,stride,extra", LOWER_CASES)
def test_explicit_lowering_and_first_layer_convolution(oracle, N, Hh, Ww, Cc, kh, kw, pad, stride, extra):
    """pipe_lower_conv_input == the lowering written out on the host, and pipe_expanded_linear on its rows == the
    oracle: the route for convolutions whose channel count the implicit form does not take."""
    rng = np.random.default_rng(N + Hh + Cc)
    x4 = rng.standard_normal((N, Hh, Ww, Cc)).astype(np.float32)
    xq4, sx = H.gpu_quantize(x4.reshape(-1, Cc))
    xq_o, sx_o = oracle.quantize_act(x4.reshape(-1, Cc))
    want_rows, Ho, Wo = _lower_im2col(xq_o.reshape(N, Hh, Ww, Cc), kh, kw, pad, pad, stride)
    I = kh * kw * Cc
    T = N * Ho * Wo
    buf = torch.full((T, I + extra), 77, dtype=torch.int8, device="cuda")
    geom = B.ConvGeom()
    geom.batch, geom.height, geom.width, geom.channels = N, Hh, Ww, Cc
    geom.kernel_h, geom.kernel_w, geom.pad_h, geom.pad_w = kh, kw, pad, pad
    geom.stride_h = geom.stride_w = stride
    B.pipe_lower_conv_input(geom, xq4.view(N, Hh, Ww, Cc), buf)
    torch.cuda.synchronize()
    got = buf.cpu().numpy()
    np.testing.assert_array_equal(got[:, :I], want_rows)
    assert (got[:, I:] == 77).all(), "bytes beyond the row were written"
    O, bits, K, g, n_keep = 64, (8 if I % 2 else 4), 3, 8, 3   # (a row of 4-bit codes is a whole number of bytes)
    W = _w(rng, O, I)
    e = oracle.expand(W, bits, K, g, n_keep)
    layer = H.gpu_expand(H.desc_of(O, I, bits, K, g, n_keep), W)
    f = oracle.forward(e, want_rows, sx_o)
    y = torch.full((T, O), float("nan"), dtype=torch.float32, device="cuda")
    B.pipe_expanded_linear(layer.desc, layer.blob, buf[:, :I], sx, y)
    torch.cuda.synchronize()
    assert B.pipe_poll_status() == B.PIPE_OK
    np.testing.assert_array_equal(y.cpu().numpy().view(np.uint32), f.y.view(np.uint32))


def test_two_layer_convolutional_ensemble_chain(oracle):
    """Sec. 3.2 / Fig. 2 on a small ConvNet: two predictors, each a chain of two convolutions on its own tensors; the
    inner layer hands Q(ReLU(y_m)) to the same predictor's next layer, the last layer's outputs are summed.  Equal, bit
    for bit, to the same composition of the oracle's pinned functions on explicitly lowered rows."""
    rng = np.random.default_rng(5)
    N, Hh, Ww, C0, C1, O, bits, K, g, M = 2, 12, 12, 128, 128, 40, 4, 4, 8, 2
    W1, W2 = _w(rng, C1, 9 * C0), _w(rng, O, 9 * C1)
    b1, b2 = rng.standard_normal(C1).astype(np.float32), rng.standard_normal(O).astype(np.float32)
    e1, e2 = oracle.expand(W1, bits, K, g, 6), oracle.expand(W2, bits, K, g, 2)
    l1 = H.gpu_expand(H.desc_of(C1, 9 * C0, bits, K, g, 6, M), W1)
    l2 = H.gpu_expand(H.desc_of(O, 9 * C1, bits, K, g, 2, M), W2)
    split = oracle.balanced_split(K, M)
    begin = np.concatenate([[0], np.cumsum(split)]).astype(int)
    x4 = np.maximum(rng.standard_normal((N, Hh, Ww, C0)), 0).astype(np.float32)
    xq4, sx = H.gpu_quantize(x4.reshape(-1, C0))
    xq_o, sx_o = oracle.quantize_act(x4.reshape(-1, C0))
    geom = B.ConvGeom()
    geom.batch, geom.height, geom.width, geom.channels = N, Hh, Ww, C0
    geom.kernel_h = geom.kernel_w = 3
    geom.pad_h = geom.pad_w = 1
    geom.stride_h = geom.stride_w = 1
    T = N * Hh * Ww
    steps = [0.04, 0.09]
    # layer 1: both predictors read the network's input; predictor m keeps its own int8 tensor
    mid = [torch.full((T, C1), 99, dtype=torch.int8, device="cuda") for _ in range(M)]
    so = [torch.tensor([s], dtype=torch.float32, device="cuda") for s in steps]
    B.pipe_ensemble_conv2d_q8(l1.desc, geom, l1.blob, [xq4.view(N, Hh, Ww, C0)] * M, [sx] * M, so, mid, torch.from_numpy(b1).cuda(), True)
    # layer 2: predictor m's tensor with its step; the outputs are summed
    y = torch.full((T, O), float("nan"), dtype=torch.float32, device="cuda")
    geom.channels = C1
    B.pipe_ensemble_conv2d(l2.desc, geom, l2.blob, [t.view(N, Hh, Ww, C1) for t in mid], so, [y], torch.from_numpy(b2).cuda(), True)
    torch.cuda.synchronize()
    assert B.pipe_poll_status() == B.PIPE_OK
    rows0, _, _ = _lower_im2col(xq_o.reshape(N, Hh, Ww, C0), 3, 3, 1, 1, 1)
    rows1 = []
    for m in range(M):
        q = oracle.forward_requantized(e1, rows0, sx_o, steps[m], int(begin[m]), int(begin[m + 1]), bias=b1 if m == 0 else None, relu=True)
        np.testing.assert_array_equal(mid[m].cpu().numpy(), q)
        rows1.append(_lower_im2col(q.reshape(N, Hh, Ww, C1), 3, 3, 1, 1, 1)[0])
    want, _ = oracle.ensemble(e2, np.stack(rows1), steps, split, bias=b2, sum_branches=True)
    np.testing.assert_array_equal(y.cpu().numpy().view(np.uint32), want.view(np.uint32))
