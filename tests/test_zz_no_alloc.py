"""pipe_expand_weights_static: the expansion for callers that cannot allocate device memory.

Some users of the library run where cudaMalloc is off limits: the host application has given the
whole GPU to its own memory pool, or an allocation (which synchronises the device) would stall the
streams that are serving requests while a layer's weights are being swapped.  For them the library
carries a fixed internal workspace.  This test calls that entry point through the C ABI twice in a
row (the second call finds the first call's leftovers in the shared workspace) and requires the
blob to be byte-identical to the one the ordinary entry point writes into caller-provided
workspace -- the expansion is integer/bit-exact work, so the tolerance is zero -- and to match the
CPU oracle's expansion.  After a warm-up call (the first call on a device may make the driver load the
module that holds the fixed array) a further call must leave the device's free memory and the
allocator's counters exactly where they were: that is the promise the entry point exists for.  It also
checks that a layer beyond the fixed size is refused.  Collected last on purpose."""
import numpy as np
import pytest
import torch

from oracle import pipe_oracle as oracle
from paper_2311_15806_b200 import binding as B
from tests import gpu_harness as H

pytestmark = pytest.mark.gpu


def _blob_sections(desc, blob):
    lay = B.pipe_layout(desc)
    out = []
    b = blob.cpu().numpy()
    for k in range(desc.num_orders):
        for off, n in [(lay.codes_off[k], lay.rows[k] * lay.canon_row_bytes), (lay.scales_off[k], lay.rows[k] * 4),
                       (lay.kept_off[k], lay.kept_groups[k] * 4), (lay.cum_off[k], (lay.num_groups + 1) * 4),
                       (lay.kcodes_off[k], lay.rows[k] * lay.kernel_row_bytes)]:
            out.append(b[off:off + n].copy())
    return out


def test_static_workspace_expansion_matches_the_ordinary_one_twice():
    H.ensure_built()
    rng = np.random.default_rng(123)
    cases = [(256, 2304, 4, 3, 8, 8), (192, 520, 2, 5, 16, 3)]   # second call: other shape, other bit-width
    for O, I, bits, K, g, n_keep in cases:
        W = (rng.standard_t(4, size=(O, I)) * 0.02).astype(np.float32)
        Wd = torch.from_numpy(W).cuda()
        desc = B.make_desc(O, I, bits, K, g, n_keep)
        lay = B.pipe_layout(desc)
        assert lay.expand_ws_bytes <= B.STATIC_SCRATCH_BYTES
        want = B.alloc_bytes(lay.blob_bytes)
        want.zero_()
        B.pipe_expand_weights(desc, Wd, want, B.alloc_bytes(lay.expand_ws_bytes))
        got = B.alloc_bytes(lay.blob_bytes)
        got.zero_()
        B.pipe_expand_weights_static(desc, Wd, got)
        torch.cuda.synchronize()
        assert B.pipe_poll_status() == B.PIPE_OK
        for a, b in zip(_blob_sections(desc, got), _blob_sections(desc, want)):
            np.testing.assert_array_equal(a, b)
        assert torch.equal(got, want)
        H.assert_expansion_matches(B.ExpandedLayer(desc, lay, got), oracle.expand(W, bits, K, g, n_keep), oracle)


def test_static_workspace_call_allocates_nothing():
    H.ensure_built()
    rng = np.random.default_rng(7)
    O_, I, bits, K, g, n_keep = 128, 640, 4, 3, 8, 4
    W = torch.from_numpy((rng.standard_normal((O_, I)) * 0.02).astype(np.float32)).cuda()
    desc = B.make_desc(O_, I, bits, K, g, n_keep)
    blob = B.alloc_bytes(B.pipe_layout(desc).blob_bytes)
    B.pipe_expand_weights_static(desc, W, blob)     # warm-up: address look-up, module load
    torch.cuda.synchronize()
    # (counters of allocation EVENTS, which a tensor freed by the garbage collector in between does not move)
    def allocation_events():
        st = torch.cuda.memory_stats()
        return st["allocation.all.allocated"], st["segment.all.allocated"]
    free0, _ = torch.cuda.mem_get_info()
    events0, reserved0 = allocation_events(), torch.cuda.memory_reserved()
    B.pipe_expand_weights_static(desc, W, blob)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0, "device memory changed across a call that must not allocate"
    assert allocation_events() == events0 and torch.cuda.memory_reserved() == reserved0
    assert B.pipe_poll_status() == B.PIPE_OK


def test_static_workspace_refuses_a_layer_that_does_not_fit():
    H.ensure_built()
    desc = B.make_desc(2048, 2048, 4, 2, 8, 16)
    lay = B.pipe_layout(desc)
    assert lay.expand_ws_bytes > B.STATIC_SCRATCH_BYTES
    W = torch.zeros((2048, 2048), dtype=torch.float32, device="cuda")
    blob = B.alloc_bytes(lay.blob_bytes)
    with pytest.raises(B.PipeError) as ei:
        B.pipe_expand_weights_static(desc, W, blob)
    assert ei.value.status == B.PIPE_ERR_WORKSPACE
