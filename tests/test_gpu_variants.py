"""The variants beside the main setting on the GPU, each bit for bit against the oracle (oracle/pipe_oracle_ext.c):
int3 / int6 weights (Sec. 4.2), A4 / A6 and asymmetric activations with the zero-point forward (Sec. 4.3), the L2
group score and the unstructured mask (Sec. 3.1)."""
import numpy as np
import pytest
import torch

from paper_2311_15806_b200 import binding as B
from tests import gpu_harness as H

pytestmark = pytest.mark.gpu


def _w(rng, O, I, heavy=False):
    W = (rng.standard_t(4, size=(O, I)) if heavy else rng.standard_normal((O, I))) * 0.02
    W *= np.exp(rng.uniform(np.log(0.5), np.log(2.0), size=(O, 1)))
    return W.astype(np.float32)


@pytest.mark.parametrize("kernel", [B.KERNEL_REFERENCE, B.KERNEL_TCGEN05, B.KERNEL_TCGEN05_PAIR, B.KERNEL_STREAM, B.KERNEL_DECODE_TC, B.KERNEL_AUTO])
@pytest.mark.parametrize("bits,O,I,T,K,g,n_keep,M", [(3, 256, 384, 300, 3, 8, 12, 1), (6, 192, 200, 270, 2, 8, 10, 2),
                                                      (3, 128, 640, 9, 4, 8, 5, 2), (6, 64, 128, 16, 2, 8, 8, 1)])
def test_int3_and_int6_layers_match_the_oracle(oracle, kernel, bits, O, I, T, K, g, n_keep, M):
    H.ensure_built()
    rng = np.random.default_rng(100 * bits + O)
    W = _w(rng, O, I)
    e = oracle.expand_ex(W, bits, K, g, n_keep)
    layer = H.gpu_expand(H.desc_of(O, I, bits, K, g, n_keep, M), W)
    H.assert_expansion_matches(layer, e, oracle)
    split = [layer.layout.branch_orders[m] for m in range(M)]
    xs = [rng.standard_normal((T, I)).astype(np.float32) for _ in range(M)]
    q = [H.gpu_quantize(x) for x in xs]
    qo = [oracle.quantize_act(x) for x in xs]
    try:
        ys, part = H.gpu_ensemble(layer, [a for a, _ in q], [b for _, b in q], None, kernel=kernel)
    except B.PipeError as ex:
        if ex.status == B.PIPE_ERR_UNSUPPORTED and kernel != B.KERNEL_AUTO:
            pytest.skip("this kernel does not take this shape")
        raise
    assert B.pipe_poll_status() == B.PIPE_OK
    want_part = np.zeros((T, e.R_total), np.int32)
    k0 = 0
    for m in range(M):
        f = oracle.forward(e, qo[m][0], qo[m][1], k0, k0 + split[m])
        np.testing.assert_array_equal(ys[m].view(np.uint32), f.y.view(np.uint32), err_msg=f"predictor {m}")
        lo, hi = e.row_off(k0), e.row_off(k0 + split[m])
        want_part[:, lo:hi] = f.partials[:, lo:hi]
        k0 += split[m]
    np.testing.assert_array_equal(part, want_part)


def _gpu_quantize_ex(x, act_bits, asym, static_scale=None, static_range=None):
    xd = torch.from_numpy(x).cuda()
    xq = torch.empty(xd.shape, dtype=torch.int8, device="cuda")
    sx = torch.zeros(1, dtype=torch.float32, device="cuda")
    zp = torch.full((1,), 99, dtype=torch.int32, device="cuda")
    ss = None if static_scale is None else torch.tensor([static_scale], dtype=torch.float32, device="cuda")
    sr = None if static_range is None else torch.tensor(static_range, dtype=torch.float32, device="cuda")
    B.pipe_quantize_act_ex(xd, xq, sx, zp, B.alloc_bytes(256), act_bits, asym, ss, sr)
    torch.cuda.synchronize()
    return xq, sx, zp


@pytest.mark.parametrize("shape", [(37, 200), (1, 17), (300, 1024)])
@pytest.mark.parametrize("act_bits,asym", [(8, False), (6, False), (4, False), (8, True), (6, True), (4, True)])
def test_activation_quantizers_match_the_oracle(oracle, shape, act_bits, asym):
    H.ensure_built()
    rng = np.random.default_rng(shape[0] + act_bits)
    x = rng.standard_normal(shape).astype(np.float32)
    if asym:
        x = np.maximum(x, -0.4).astype(np.float32) * 3      # skewed range
    xq, sx, zp = _gpu_quantize_ex(x, act_bits, asym)
    want_q, want_s, want_z = oracle.quantize_act_ex(x, act_bits, asym)
    assert B.pipe_poll_status() == B.PIPE_OK
    assert np.float32(sx.item()).view(np.uint32) == np.float32(want_s).view(np.uint32)
    assert int(zp.item()) == want_z
    np.testing.assert_array_equal(xq.cpu().numpy(), want_q)
    # static step / static range (values clamp)
    if asym:
        rng_ = (float(x.min()) * 0.5, float(x.max()) * 0.5)
        xq, sx, zp = _gpu_quantize_ex(x, act_bits, True, static_range=rng_)
        want_q, want_s, want_z = oracle.quantize_act_ex(x, act_bits, True, static_range=rng_)
    else:
        step = float(np.abs(x).max()) / 40
        xq, sx, zp = _gpu_quantize_ex(x, act_bits, False, static_scale=step)
        want_q, want_s, want_z = oracle.quantize_act_ex(x, act_bits, False, static_scale=step)
    assert np.float32(sx.item()).view(np.uint32) == np.float32(want_s).view(np.uint32) and int(zp.item()) == want_z
    np.testing.assert_array_equal(xq.cpu().numpy(), want_q)


def test_activation_quantizer_edge_cases(oracle):
    H.ensure_built()
    zeros = np.zeros((3, 8), np.float32)
    for asym in (False, True):
        xq, sx, zp = _gpu_quantize_ex(zeros, 8, asym)
        assert sx.item() == 0.0 and zp.item() == 0 and not xq.cpu().numpy().any()
    bad = zeros.copy()
    bad[1, 2] = np.nan
    _gpu_quantize_ex(bad, 6, True)
    assert B.pipe_poll_status() == B.PIPE_ERR_NONFINITE
    x = np.ones((2, 8), np.float32)
    xd = torch.from_numpy(x).cuda()
    with pytest.raises(B.PipeError):   # a static step has no meaning for the asymmetric quantizer
        B.pipe_quantize_act_ex(xd, torch.empty((2, 8), dtype=torch.int8, device="cuda"), torch.zeros(1, device="cuda"),
                               torch.zeros(1, dtype=torch.int32, device="cuda"), B.alloc_bytes(256), 8, True,
                               torch.ones(1, device="cuda"), None)
    with pytest.raises(B.PipeError):
        B.pipe_quantize_act_ex(xd, torch.empty((2, 8), dtype=torch.int8, device="cuda"), torch.zeros(1, device="cuda"),
                               torch.zeros(1, dtype=torch.int32, device="cuda"), B.alloc_bytes(256), 5, False)


@pytest.mark.parametrize("O,I,T,bits,K,g,n_keep,M", [(64, 100, 70, 4, 3, 8, 4, 1), (128, 256, 130, 2, 4, 16, 3, 2),
                                                      (72, 260, 33, 8, 2, 8, 9, 2)])
def test_zero_point_forward_matches_the_oracle(oracle, O, I, T, bits, K, g, n_keep, M):
    H.ensure_built()
    rng = np.random.default_rng(O + T)
    W = _w(rng, O, I, heavy=(bits == 2))
    bias = rng.standard_normal(O).astype(np.float32) * 0.1
    e = oracle.expand_ex(W, bits, K, g, n_keep)
    layer = H.gpu_expand(H.desc_of(O, I, bits, K, g, n_keep, M), W)
    split = [layer.layout.branch_orders[m] for m in range(M)]
    xs = [(np.maximum(rng.standard_normal((T, I)), -0.3) * (1 + m)).astype(np.float32) for m in range(M)]
    q = [_gpu_quantize_ex(x, 8, True) for x in xs]
    qo = [oracle.quantize_act_ex(x, 8, True) for x in xs]
    ys = [torch.full((T, O), float("nan"), dtype=torch.float32, device="cuda") for _ in range(M)]
    part = torch.zeros((T, e.R_total), dtype=torch.int32, device="cuda")
    B.pipe_ensemble_forward_zp(layer.desc, layer.blob, [a for a, _, _ in q], [b for _, b, _ in q], [c for _, _, c in q], ys,
                               torch.from_numpy(bias).cuda(), False, part)
    torch.cuda.synchronize()
    assert B.pipe_poll_status() == B.PIPE_OK
    want_part = np.zeros((T, e.R_total), np.int32)
    k0 = 0
    for m in range(M):
        assert qo[m][2] != 0          # the case does exercise a zero point
        f, _ = oracle.forward_zp(e, qo[m][0], qo[m][1], qo[m][2], k0, k0 + split[m], bias=bias if m == 0 else None)
        np.testing.assert_array_equal(ys[m].cpu().numpy().view(np.uint32), f.y.view(np.uint32), err_msg=f"predictor {m}")
        lo, hi = e.row_off(k0), e.row_off(k0 + split[m])
        want_part[:, lo:hi] = f.partials[:, lo:hi]
        k0 += split[m]
    np.testing.assert_array_equal(part.cpu().numpy(), want_part)
    # the tensor-core kernels decline the zero point instead of ignoring it
    B.pipe_diag_select_kernel(B.KERNEL_TCGEN05)
    try:
        with pytest.raises(B.PipeError) as ei:
            B.pipe_ensemble_forward_zp(layer.desc, layer.blob, [a for a, _, _ in q], [b for _, b, _ in q], [c for _, _, c in q], ys)
        assert ei.value.status == B.PIPE_ERR_UNSUPPORTED
    finally:
        B.pipe_diag_select_kernel(B.KERNEL_AUTO)


@pytest.mark.parametrize("O,I,bits,K,g,n_keep", [(256, 300, 4, 3, 8, 9), (4800, 64, 2, 3, 8, 150), (128, 1000, 8, 2, 16, 3)])
def test_l2_group_score_matches_the_oracle(oracle, O, I, bits, K, g, n_keep):
    H.ensure_built()
    rng = np.random.default_rng(O + I)
    W = (_w(rng, O, I) * np.exp(rng.uniform(-1.5, 1.5, size=(O, 1)))).astype(np.float32)
    e = oracle.expand_ex(W, bits, K, g, n_keep, score_mode=oracle.SCORE_L2)
    e0 = oracle.expand_ex(W, bits, K, g, n_keep)
    assert any((e.order_kept(k) != e0.order_kept(k)).any() for k in range(1, K))   # the two scores do pick different groups here
    d = B.make_desc(O, I, bits, K, g, n_keep, 1, None, B.SCORE_L2)
    layer = H.gpu_expand(d, W)
    H.assert_expansion_matches(layer, e, oracle)


@pytest.mark.parametrize("O,I,bits,K,g,keep_elems", [(64, 333, 4, 3, 8, 40), (24, 2048, 2, 4, 8, 512), (16, 100, 8, 2, 4, 1),
                                                      (8, 64, 4, 3, 8, 64)])
def test_unstructured_mask_matches_the_oracle(oracle, O, I, bits, K, g, keep_elems):
    H.ensure_built()
    rng = np.random.default_rng(O * I)
    W = _w(rng, O, I, heavy=True)
    W[0, : I // 2] = W[0, 0]          # a row full of ties: the lower indices win
    I_eff = I - I % (8 // (2 if bits == 2 else (4 if bits <= 4 else 8)))
    W = W[:, :I_eff]
    keep_elems = min(keep_elems, I_eff)
    G = O // g
    e = oracle.expand_ex(W, bits, K, g, G, elem_keep=keep_elems)
    d = B.make_desc(O, I_eff, bits, K, g, G, 1, None, B.SCORE_MAXABS, keep_elems)
    layer = H.gpu_expand(d, W)
    H.assert_expansion_matches(layer, e, oracle)
    for k in range(1, K):
        assert (np.count_nonzero(e.order_codes(k), axis=1) <= keep_elems).all()
    # the masked layer runs through the ordinary forward (its orders are full-height tensors with zeros in them)
    x = rng.standard_normal((20, I_eff)).astype(np.float32)
    xq, sx = H.gpu_quantize(x)
    xo, so = oracle.quantize_act(x)
    y, part = H.gpu_linear(layer, xq, sx)
    f = oracle.forward(e, xo, so)
    np.testing.assert_array_equal(part, f.partials)
    np.testing.assert_array_equal(y.view(np.uint32), f.y.view(np.uint32))


@pytest.mark.parametrize("kernel", [B.KERNEL_REFERENCE, B.KERNEL_TCGEN05, B.KERNEL_TCGEN05_PAIR, B.KERNEL_STREAM, B.KERNEL_DECODE_TC, B.KERNEL_AUTO])
@pytest.mark.parametrize("act", [B.ACT_SILU, B.ACT_GELU, B.ACT_SIGMOID])
def test_smooth_activations_in_the_fused_epilogue(oracle, kernel, act):
    """Inner layer with SiLU / GeLU / sigmoid (Sec. 3.2): the oracle evaluates sigma in binary64 and rounds once, the
    kernels evaluate it in binary32 with the device's exp / erf, so a code on a rounding boundary may come out one
    step off -- the tolerance is one code, on at most half a percent of the outputs; the integer sums stay exact."""
    H.ensure_built()
    rng = np.random.default_rng(act)
    O, I, T, bits, K, g, n_keep, M = 192, 256, 300 if kernel not in (B.KERNEL_STREAM, B.KERNEL_DECODE_TC) else 16, 4, 4, 8, 12, 2
    W = _w(rng, O, I)
    bias = rng.standard_normal(O).astype(np.float32) * 0.1
    e = oracle.expand(W, bits, K, g, n_keep)
    layer = H.gpu_expand(H.desc_of(O, I, bits, K, g, n_keep, M), W)
    split = [layer.layout.branch_orders[m] for m in range(M)]
    xs = [rng.standard_normal((T, I)).astype(np.float32) for _ in range(M)]
    q = [H.gpu_quantize(x) for x in xs]
    qo = [oracle.quantize_act(x) for x in xs]
    steps, want = [], []
    k0 = 0
    for m in range(M):
        fm = oracle.forward(e, qo[m][0], qo[m][1], k0, k0 + split[m], bias=bias if m == 0 else None)
        a = oracle.activation(fm.y, act)
        s = float(np.float32(np.quantile(np.abs(a), 0.97) / 127 + 1e-12))
        steps.append(s)
        want.append(oracle.quantize_act(a, static_scale=s)[0])
        k0 += split[m]
    try:
        got, _ = H.gpu_ensemble_q8(layer, [a for a, _ in q], [b for _, b in q], steps, bias, relu=act, kernel=kernel, want_partials=False)
    except B.PipeError as ex:
        if ex.status == B.PIPE_ERR_UNSUPPORTED and kernel != B.KERNEL_AUTO:
            pytest.skip("this kernel does not take this shape")
        raise
    assert B.pipe_poll_status() == B.PIPE_OK
    for m in range(M):
        diff = np.abs(got[m].astype(np.int32) - want[m].astype(np.int32))
        assert diff.max() <= 1
        assert (diff != 0).mean() <= 0.005
