"""Diagnostic entry points (include/pipe_diag.h) on the GPU: the bounded wait of the kernels runs out the
way it is documented to -- PIPE_ERR_TIMEOUT in the status word, a normal return, a usable device -- and the
issue-rate probe of the integer tensor pipe runs and reports a plausible rate."""
import numpy as np
import pytest
import torch

from oracle import pipe_oracle as O
from paper_2311_15806_b200 import binding as B
from tests import gpu_harness as H

pytestmark = pytest.mark.gpu


def test_bounded_wait_runs_out_and_leaves_the_device_usable():
    H.ensure_built()
    torch.cuda.synchronize()
    assert B.pipe_poll_status() == B.PIPE_OK
    B.pipe_diag_bounded_wait(20000)          # a barrier nobody arrives on; the wait gives up after 20 k cycles
    torch.cuda.synchronize()                 # the kernel returned by itself
    assert B.pipe_poll_status() == B.PIPE_ERR_TIMEOUT
    assert B.pipe_poll_status() == B.PIPE_OK  # the poll cleared the word
    # the context is intact: an ordinary call still gives the oracle's answer
    x = np.random.default_rng(5).standard_normal((37, 200)).astype(np.float32)
    xq, sx = H.gpu_quantize(x)
    want_q, want_s = O.quantize_act(x)
    np.testing.assert_array_equal(xq.cpu().numpy(), want_q)
    assert np.float32(sx.item()).view(np.uint32) == np.float32(want_s).view(np.uint32)
    assert B.pipe_poll_status() == B.PIPE_OK


def test_bounded_wait_rejects_bad_limits():
    H.ensure_built()
    for bad in (0, -5, 1 << 40):
        with pytest.raises(B.PipeError) as ei:
            B.pipe_diag_bounded_wait(bad)
        assert ei.value.status == B.PIPE_ERR_INVALID_ARG


@pytest.mark.parametrize("n_cols", [64, 256])
def test_integer_tensor_pipe_probe(n_cols):
    H.ensure_built()
    B.pipe_diag_mma_i8_rate(n_cols, 512)     # warm-up
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    ops = B.pipe_diag_mma_i8_rate(n_cols, 20000)
    e1.record()
    torch.cuda.synchronize()
    assert B.pipe_poll_status() == B.PIPE_OK
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    assert ops == 2.0 * 128 * n_cols * 32 * 20000 * sms
    tops = ops / (e0.elapsed_time(e1) * 1e-3) / 1e12
    # nominal dense int8 rate of the part is 4500 TOP/s; a working probe lands within a factor of a few below it
    assert 500.0 < tops < 6000.0, tops
    with pytest.raises(B.PipeError):
        B.pipe_diag_mma_i8_rate(100, 10)
