"""The five benchmark configurations at full size, in the launch configuration bench.py times
(paper_2311_15806_b200.runner.LayerRunner, automatic kernel choice).

Weight expansion is compared with the oracle in full (every code, scale and kept list).  The
contraction is too large for the CPU at these sizes, so int32 partial sums and fp32 outputs are
compared on sampled token rows (first/last rows, both sides of tile boundaries, seeded random rows)
for ALL output channels and orders; between the samples the tensor-core kernel is cross-checked in
full against the CUDA-core kernel, which shares neither its code layout nor its tiling.  The inner-layer
form (int8 output) is checked the same way: sampled rows against the oracle, every element against the
quantizer kernel applied to the pinned fp32 output."""
import numpy as np
import pytest
import torch

from paper_2311_15806_b200 import binding as B
from paper_2311_15806_b200 import synth
from paper_2311_15806_b200.runner import LayerRunner
from tests import gpu_harness as H

pytestmark = pytest.mark.gpu

WORK = synth.paper_workloads()
N_SAMPLE = 72


@pytest.fixture(scope="module", autouse=True)
def _built():
    H.ensure_built()


def _check_layer(oracle, spec, token_counts=None, second_layer=False, cross_check=True, int8_copy=False):
    run = LayerRunner(spec, second_layer=second_layer, int8_copy=int8_copy)
    W = run.host_weights()
    e = oracle.expand(W, spec.bits, spec.K, spec.g, run.n_keep)
    split = [int(v) for v in oracle.balanced_split(spec.K, spec.M)]
    first = True
    for T in (token_counts or [spec.T]):
        sp = spec.with_tokens(T) if spec.conv is None else spec
        run.spec = sp
        if sp.conv is not None:
            x4 = [synth.make_conv_input(sp, m) for m in range(sp.M if run.distinct_inputs else 1)]
            run.load(W)
            rows = synth.sample_rows(run.T, N_SAMPLE, 128, sp.seed)
            xs_rows = [synth.im2col_rows(x, sp.conv, rows) for x in x4]
            sx_full = [oracle.quantize_act(x.reshape(-1, x.shape[-1]))[1] for x in x4]
        else:
            xs = [synth.make_activations(sp, m) for m in range(sp.M if run.distinct_inputs else 1)]
            run.load(W, xs)
            rows = synth.sample_rows(run.T, N_SAMPLE, 128, sp.seed)
            xs_rows = [x[rows] for x in xs]
            sx_full = [oracle.quantize_act(x)[1] for x in xs]
        part = torch.zeros((run.T, run.total_rows), dtype=torch.int32, device="cuda")
        run.expand()
        run.quantize()
        run.forward(part)
        torch.cuda.synchronize()
        assert B.pipe_poll_status() == B.PIPE_OK
        if first:
            H.assert_expansion_matches(run.layer, e, oracle)
            first = False
        rows_t = torch.from_numpy(rows).cuda()
        k0 = 0
        for m in range(sp.M):
            i = m if len(xs_rows) > 1 else 0
            assert run.sx[i].cpu().numpy().view(np.uint32)[0] == np.float32(sx_full[i]).view(np.uint32)
            xq_o, _ = oracle.quantize_act(xs_rows[i], static_scale=float(sx_full[i]))
            if run.geom is None:
                np.testing.assert_array_equal(run.xq[i][rows_t].cpu().numpy(), xq_o)
            else:   # implicit convolution: the quantized tensor is the NHWC input itself
                x_nhwc = x4[i].reshape(-1, x4[i].shape[-1])
                np.testing.assert_array_equal(run.xq[i].cpu().numpy(), oracle.quantize_act(x_nhwc)[0])
            f = oracle.forward(e, xq_o, sx_full[i], k0, k0 + split[m])
            lo, hi = e.row_off(k0), e.row_off(k0 + split[m])
            np.testing.assert_array_equal(part[rows_t][:, lo:hi].cpu().numpy(), f.partials[:, lo:hi])
            y = run.y[m][rows_t].cpu().numpy()
            H.assert_outputs_close(y, f, f"{sp.name} T={run.T} branch {m}")
            np.testing.assert_array_equal(y.view(np.uint32), f.y.view(np.uint32))
            k0 += split[m]
        # inner-layer form of the same launch (activation function and the next layer's input quantizer fused into
        # the epilogue): the oracle on the sampled rows, and every element against ReLU + the quantizer kernel
        # applied to the fp32 output that the lines above have just pinned
        steps = [(y.clamp_min(0).max() * (0.5 / 127)).reshape(1).float() for y in run.y]
        yq = run.forward_q8(steps, relu=True)
        torch.cuda.synchronize()
        assert B.pipe_poll_status() == B.PIPE_OK
        k0 = 0
        for m in range(sp.M):
            i = m if len(xs_rows) > 1 else 0
            step = float(steps[m].cpu())
            xq_o, _ = oracle.quantize_act(xs_rows[i], static_scale=float(sx_full[i]))
            want = oracle.forward_requantized(e, xq_o, sx_full[i], step, k0, k0 + split[m], relu=True)
            np.testing.assert_array_equal(yq[m][rows_t].cpu().numpy(), want)
            assert int(yq[m].max()) == 127 and int(yq[m].min()) == 0     # the step clamps the largest outputs; ReLU
            a = run.y[m].clamp_min(0)
            full, _ = H.gpu_quantize(None, static_scale=step, xd=a)
            assert torch.equal(yq[m], full)
            del a, full
            k0 += split[m]
        del yq
        if hasattr(run, "yq"):
            del run.yq
        torch.cuda.empty_cache()
        if run.geom is not None:
            # implicit GEMM vs the same layer on explicitly lowered rows (and that one vs the CUDA-core kernel)
            y_conv = run.y[0].clone()
            part_conv = part.clone()
            del run
            torch.cuda.empty_cache()
            run = LayerRunner(sp, implicit_conv=False)
            run.load(W)
            run.expand()
            run.quantize()
            part.zero_()
            run.forward(part)
            torch.cuda.synchronize()
            assert torch.equal(y_conv.view(torch.int32), run.y[0].view(torch.int32))
            assert torch.equal(part_conv, part)
            del y_conv, part_conv
        if cross_check:
            # the whole output, tensor-core/streaming kernel vs CUDA-core kernel, bit for bit
            y_auto = [y.clone() for y in run.y]
            part_auto = part.clone()
            part.zero_()
            B.pipe_diag_select_kernel(B.KERNEL_REFERENCE)
            try:
                run.forward(part)
                torch.cuda.synchronize()
            finally:
                B.pipe_diag_select_kernel(B.KERNEL_AUTO)
            for m in range(sp.M):
                assert torch.equal(y_auto[m].view(torch.int32), run.y[m].view(torch.int32))
            assert torch.equal(part_auto, part)
        del part
        torch.cuda.empty_cache()


def test_cfg1_int8_dense(oracle):
    _check_layer(oracle, WORK["cfg1"])


def test_cfg2_conv_int4(oracle):
    _check_layer(oracle, WORK["cfg2"])


def test_cfg3_bert_ffn_int4(oracle):
    _check_layer(oracle, WORK["cfg3a"])
    _check_layer(oracle, WORK["cfg3b"], second_layer=True)


def test_cfg4_llm_mlp_up_projection(oracle):
    _check_layer(oracle, WORK["cfg4a_t1"], token_counts=[1, 16, 128, 1024, 4096])


def test_cfg4_llm_mlp_down_projection(oracle):
    _check_layer(oracle, WORK["cfg4b_t1"], token_counts=[1, 16, 128, 1024, 4096], second_layer=True)


def test_cfg5_ternary(oracle):
    _check_layer(oracle, WORK["cfg5"], cross_check=False)


def test_cfg5_ternary_cross_check_on_a_token_slice(oracle):
    """The CUDA-core kernel needs seconds for the full 1.5e12 MACs; cross-check 1024 tokens."""
    _check_layer(oracle, WORK["cfg5"].with_tokens(1024), cross_check=True)


def test_layers_with_an_int8_copy_at_full_size(oracle):
    """The rows bench.py measures once more on layers that keep the int8 copy of their codes: same checks, same bits."""
    _check_layer(oracle, WORK["cfg3a"], int8_copy=True)
    _check_layer(oracle, WORK["cfg3b"], second_layer=True, int8_copy=True)
    _check_layer(oracle, WORK["cfg4a_t1"], token_counts=[16, 128, 1024, 4096], int8_copy=True)
    _check_layer(oracle, WORK["cfg4b_t1"], token_counts=[4096], second_layer=True, int8_copy=True)
