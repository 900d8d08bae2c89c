"""The C-ABI library: it loads without a GPU, exports every symbol the header declares, and its
host-side logic (descriptor validation, blob layout, splits, kept-group counts) is right."""
import ctypes as C
import os
import re

import pytest

from paper_2311_15806_b200 import binding as B
from paper_2311_15806_b200 import build as pipe_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    pipe_build.build()
    return B.lib()


def _declared_functions():
    names = set()
    for header in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if not header.endswith(".h"):
            continue
        text = open(os.path.join(ROOT, "include", header)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names.update(re.findall(r"\b(pipe_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_every_declared_symbol_is_exported(lib):
    names = _declared_functions()
    assert len(names) >= 11
    for n in names:
        assert hasattr(lib, n), n
    assert set(B.EXPORTS) == set(names)


def test_status_strings(lib):
    assert B.pipe_status_string(0) == "ok"
    assert len({B.pipe_status_string(s) for s in range(10)}) == 10


def test_keep_groups_and_default_branches(lib):
    assert B.pipe_keep_groups_from_gamma(32, 0.25) == 8
    assert B.pipe_keep_groups_from_gamma(1376, 0.5) == 688
    assert B.pipe_keep_groups_from_gamma(10, 0.33) == 4
    assert B.pipe_keep_groups_from_gamma(10, 0.0) == 1 and B.pipe_keep_groups_from_gamma(10, 3.0) == 10
    with open(os.path.join(ROOT, "tests", "golden", "ensemble_splits.txt")) as f:
        for line in f:
            line = line.split("#")[0].split()
            if line:
                assert B.pipe_default_branches(int(line[0]), int(line[1])) == [int(v) for v in line[2].split(",")]
    with pytest.raises(B.PipeError):
        B.pipe_default_branches(2, 3)


def test_layout_sections_are_disjoint_and_aligned(lib):
    d = B.make_desc(256, 2304, 4, 3, 8, 8, 1)
    lay = B.pipe_layout(d)
    assert lay.num_groups == 32 and lay.total_rows == 256 + 2 * 64
    assert lay.canon_row_bytes == 1152 and lay.kernel_row_bytes == 1152
    assert [lay.rows[k] for k in range(3)] == [256, 64, 64]
    spans = []
    for k in range(3):
        spans += [(lay.codes_off[k], lay.rows[k] * lay.canon_row_bytes), (lay.scales_off[k], lay.rows[k] * 4),
                  (lay.kept_off[k], lay.kept_groups[k] * 4), (lay.cum_off[k], 33 * 4),
                  (lay.kcodes_off[k], lay.rows[k] * lay.kernel_row_bytes)]
        assert lay.kcodes_off[k] % 1024 == 0 and lay.codes_off[k] % 256 == 0
    spans.sort()
    assert spans[0][0] >= 1024
    for (o0, n0), (o1, _) in zip(spans, spans[1:]):
        assert o0 + n0 <= o1
    assert spans[-1][0] + spans[-1][1] <= lay.blob_bytes
    # ragged reduction length: kernel rows are padded to 128 codes
    lay2 = B.pipe_layout(B.make_desc(16, 200, 2, 2, 4, 2, 2))
    assert lay2.canon_row_bytes == 50 and lay2.kernel_row_bytes == 64
    assert [lay2.branch_orders[m] for m in range(2)] == [1, 1]
    assert lay2.expand_ws_bytes >= 16 * 200 * 4


def test_layout_with_an_int8_copy(lib):
    plain = B.pipe_layout(B.make_desc(256, 2300, 4, 3, 8, 8, 1))
    assert all(plain.wcodes_off[k] == 0 for k in range(16))
    d = B.make_desc(256, 2300, 4, 3, 8, 8, 1, int8_copy=True)
    lay = B.pipe_layout(d)
    ipad = 2304
    spans = []
    for k in range(3):
        assert lay.wcodes_off[k] % 1024 == 0 and lay.wcodes_off[k] > 0
        spans += [(lay.codes_off[k], lay.rows[k] * lay.canon_row_bytes), (lay.scales_off[k], lay.rows[k] * 4),
                  (lay.kept_off[k], lay.kept_groups[k] * 4), (lay.cum_off[k], 33 * 4),
                  (lay.kcodes_off[k], lay.rows[k] * lay.kernel_row_bytes), (lay.wcodes_off[k], lay.rows[k] * ipad)]
    spans += [(lay.blk_off[m], 4 * (lay.blk_cap[m] + 2)) for m in range(2)]
    spans += [(lay.rec_off[m], B.BLOCK_RECORD_BYTES * lay.rec_cap[m]) for m in range(2)]
    spans.sort()
    for (o0, n0), (o1, _) in zip(spans, spans[1:]):
        assert o0 + n0 <= o1
    assert spans[-1][0] + spans[-1][1] <= lay.blob_bytes
    assert lay.blob_bytes >= plain.blob_bytes + sum(lay.rows[k] for k in range(3)) * ipad
    # the copy keeps 8-row atoms whole, so the group size must be a multiple of 8; the flag is 0 or 1
    bad = B.make_desc(256, 2304, 4, 3, 4, 8, 1, int8_copy=True)
    with pytest.raises(B.PipeError) as ex:
        B.pipe_layout(bad)
    assert ex.value.status == B.PIPE_ERR_SHAPE
    bad = B.make_desc(256, 2304, 4, 3, 8, 8, 1)
    bad.int8_copy = 2
    with pytest.raises(B.PipeError) as ex:
        B.pipe_layout(bad)
    assert ex.value.status == B.PIPE_ERR_INVALID_ARG


@pytest.mark.parametrize("kwargs,status", [
    (dict(O=0), B.PIPE_ERR_INVALID_ARG), (dict(bits=5), B.PIPE_ERR_INVALID_ARG), (dict(K=17), B.PIPE_ERR_INVALID_ARG),
    (dict(g=7), B.PIPE_ERR_SHAPE), (dict(keep=0), B.PIPE_ERR_INVALID_ARG), (dict(keep=9), B.PIPE_ERR_INVALID_ARG),
    (dict(M=5), B.PIPE_ERR_SHAPE), (dict(I=63, bits=4), B.PIPE_ERR_SHAPE), (dict(I=133200, bits=8), B.PIPE_ERR_ACC_OVERFLOW),
    (dict(branch=[3, 2]), B.PIPE_ERR_SHAPE), (dict(branch=[4, 0]), B.PIPE_ERR_SHAPE),
])
def test_bad_descriptors_are_rejected(lib, kwargs, status):
    a = dict(O=64, I=64, bits=4, K=4, g=8, keep=4, M=2, branch=None)
    a.update(kwargs)
    d = B.make_desc(a["O"], a["I"], a["bits"], a["K"], a["g"], a["keep"], a["M"], a["branch"])
    with pytest.raises(B.PipeError) as ei:
        B.pipe_layout(d)
    assert ei.value.status == status


@pytest.mark.parametrize("bits,last_ok", [(8, 133144), (4, 150976), (2, 264208)])
def test_accumulator_bound_sits_where_the_scaled_codes_put_it(lib, bits, last_ok):
    # the kernels hold sub-byte codes as code * 2^(8-b): 127 * qmax * 2^(8-b) * I must stay below 2^31
    qmax = (1 << (bits - 1)) - 1
    per_byte = 8 // bits
    ok = last_ok // per_byte * per_byte
    bad = ok + per_byte
    assert 127 * qmax * (1 << (8 - bits)) * ok < 2 ** 31 <= 127 * qmax * (1 << (8 - bits)) * (last_ok + 1)
    B.pipe_layout(B.make_desc(8, ok, bits, 1, 8, 1, 1))
    with pytest.raises(B.PipeError) as ei:
        B.pipe_layout(B.make_desc(8, bad, bits, 1, 8, 1, 1))
    assert ei.value.status == B.PIPE_ERR_ACC_OVERFLOW


def test_explicit_branch_orders(lib):
    lay = B.pipe_layout(B.make_desc(64, 64, 4, 4, 8, 4, 2, [3, 1]))
    assert [lay.branch_orders[m] for m in range(2)] == [3, 1]


def test_compute_calls_validate_before_touching_the_device(lib):
    d = B.make_desc(64, 64, 4, 2, 8, 4, 1)
    lay = B.pipe_layout(d)
    # null pointers / undersized buffers are host-detectable and must not reach CUDA
    assert lib.pipe_expand_weights(C.byref(d), None, 64, None, 0, None, 0, None) == B.PIPE_ERR_INVALID_ARG
    assert lib.pipe_expand_weights(C.byref(d), 4096, 64, 8192, 16, 4096, 16, None) == B.PIPE_ERR_WORKSPACE
    assert lib.pipe_expand_weights(C.byref(d), 4096, 64, 8192 + 8, lay.blob_bytes, 4096, lay.expand_ws_bytes,
                                   None) == B.PIPE_ERR_ALIGNMENT
    assert lib.pipe_quantize_act(None, 4, 64, 64, None, None, 64, None, None, 0, None) == B.PIPE_ERR_INVALID_ARG
    assert lib.pipe_quantize_act(4096, 4, 64, 32, None, 4096, 64, 4096, 4096, 256, None) == B.PIPE_ERR_INVALID_ARG
    assert lib.pipe_expanded_linear(C.byref(d), None, None, 4, 64, None, None, None, 64, None, None) == B.PIPE_ERR_INVALID_ARG
    assert lib.pipe_diag_select_kernel(9) == B.PIPE_ERR_INVALID_ARG
    assert lib.pipe_diag_select_kernel(0) == B.PIPE_OK
