"""Stream order between the expansion and the forward kernels.

The forward kernels start under programmatic stream serialization and the weight-streaming kernel copies packed codes
ahead of its dependency wait; a forward call queued directly behind an expansion on the same stream must nevertheless
see that expansion's blob.  The weights change between rounds and nothing synchronizes inside a round, so a forward
that read the blob too early would return the previous round's outputs."""
import numpy as np
import pytest
import torch

from paper_2311_15806_b200 import binding as B
from tests import gpu_harness as H

pytestmark = pytest.mark.gpu

CASES = [
    # O, I, T, bits, K, g, n_keep, M
    (1024, 1024, 1, 4, 3, 8, 32, 1),       # weight-streaming kernel
    (1024, 1024, 16, 8, 2, 8, 64, 2),
    (768, 1024, 200, 4, 3, 8, 24, 1),      # SM-pair kernel
]


@pytest.mark.parametrize("O,I,T,bits,K,g,n_keep,M", CASES)
def test_forward_directly_behind_an_expansion_sees_its_blob(oracle, O, I, T, bits, K, g, n_keep, M):
    rng = np.random.default_rng(11 * O + T)
    d = H.desc_of(O, I, bits, K, g, n_keep, M)
    lay = B.pipe_layout(d)
    blob = B.alloc_bytes(lay.blob_bytes, "cuda")
    ws = B.alloc_bytes(lay.expand_ws_bytes, "cuda")
    x = rng.standard_normal((T, I)).astype(np.float32)
    xq, sx = H.gpu_quantize(x)
    xq_o, sx_o = oracle.quantize_act(x)
    Ws = [(rng.standard_normal((O, I)) * (0.05 * (r + 1))).astype(np.float32) for r in range(4)]
    Wd = [torch.from_numpy(w).cuda() for w in Ws]
    ys = [torch.full((T, O), float("nan"), dtype=torch.float32, device="cuda") for _ in Ws]
    torch.cuda.synchronize()
    zp = [torch.zeros(1, dtype=torch.int32, device="cuda") for _ in range(M)]
    scratch_y = [torch.empty((T, O), dtype=torch.float32, device="cuda") for _ in range(M)]
    for r in range(len(Ws)):
        B.pipe_expand_weights(d, Wd[r], blob, ws)
        if r % 2 == 1:
            # a forward call that is refused after it has looked at its arguments (a zero point with a back end forced
            # that takes none) queues nothing, so it must not count as "something stands behind the expansion now"
            B.pipe_diag_select_kernel(B.KERNEL_STREAM)
            try:
                with pytest.raises(B.PipeError) as ex:
                    B.pipe_ensemble_forward_zp(d, blob, [xq] * M, [sx] * M, zp, scratch_y, None, False, None)
                assert ex.value.status == B.PIPE_ERR_UNSUPPORTED
            finally:
                B.pipe_diag_select_kernel(B.KERNEL_AUTO)
        if M == 1:
            B.pipe_expanded_linear(d, blob, xq, sx, ys[r], None, None)
        else:
            B.pipe_ensemble_forward(d, blob, [xq] * M, [sx] * M, [ys[r]], None, True, None)
    torch.cuda.synchronize()
    assert B.pipe_poll_status() == B.PIPE_OK
    split = [lay.branch_orders[m] for m in range(M)]
    for r, W in enumerate(Ws):
        e = oracle.expand(W, bits, K, g, n_keep)
        if M == 1:
            want = oracle.forward(e, xq_o, sx_o).y
        else:
            want, _ = oracle.ensemble(e, np.stack([xq_o] * M), [sx_o] * M, split, sum_branches=True)
        np.testing.assert_array_equal(ys[r].cpu().numpy().view(np.uint32), want.view(np.uint32), err_msg=f"round {r}")
