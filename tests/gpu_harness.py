"""Helpers for the GPU parity tests: run the CUDA library through its C ABI binding and compare
with the CPU oracle.  The expected values always come from the oracle, never from the GPU."""
from __future__ import annotations

import numpy as np
import torch

from paper_2311_15806_b200 import binding as B
from paper_2311_15806_b200 import build as pipe_build

REL_TOL = 1e-5  # fp32 outputs: |y - y64| <= REL_TOL * sum_k |term_k|  (the stated output tolerance)


def ensure_built():
    pipe_build.build()
    B.lib()


INT8_COPY_DEFAULT = False   # tests/test_gpu_int8_copy.py runs other modules' cases with this switched on


def desc_of(O, I, bits, K, g, n_keep, M=1, branch_orders=None, int8_copy=None):
    if int8_copy is None:
        int8_copy = INT8_COPY_DEFAULT and g % 8 == 0
    return B.make_desc(O, I, bits, K, g, n_keep, M, branch_orders, int8_copy=int8_copy)


def gpu_expand(desc, W: np.ndarray) -> B.ExpandedLayer:
    Wd = torch.from_numpy(W).cuda()
    layer = B.expand(desc, Wd)
    torch.cuda.synchronize()
    assert B.pipe_poll_status() == B.PIPE_OK
    return layer


def kernel_layout_from_codes(codes: np.ndarray, bits: int) -> np.ndarray:
    """The documented streaming layout computed from int8 codes [rows, I] (see include/pipe.h)."""
    rows, I = codes.shape
    Ipad = (I + 127) // 128 * 128
    c = np.zeros((rows, Ipad), np.int8)
    c[:, :I] = codes
    nblk = Ipad // 128

    def block_major(packed):   # [rows, Ipad*bits/8] -> [Ipad/128, rows, 128*bits/8] flattened back to 2-D
        return np.ascontiguousarray(packed.reshape(rows, nblk, -1).transpose(1, 0, 2)).reshape(rows, -1)

    if bits == 8:
        return block_major(c.view(np.uint8))
    per_word = 32 // bits
    u = (c.astype(np.int32) & ((1 << bits) - 1)).astype(np.uint32).reshape(rows, Ipad // per_word, per_word // 4, 4)
    word = np.zeros((rows, Ipad // per_word), np.uint32)
    for h in range(per_word // 4):
        for j in range(4):
            shift = (4 * (2 * j + h)) if bits == 4 else (8 * j + 2 * h)
            word |= u[:, :, h, j] << np.uint32(shift)
    return block_major(word.view(np.uint8).reshape(rows, -1))


def assert_expansion_matches(layer: B.ExpandedLayer, e, oracle, check_kernel_layout=True):
    """Bit-exact: kept lists, prefix counts, canonical packed codes, scales, streaming layout."""
    lay = layer.layout
    assert lay.total_rows == e.R_total
    for k in range(e.K):
        kept = layer.kept(k).cpu().numpy()
        np.testing.assert_array_equal(kept, e.order_kept(k), err_msg=f"kept groups, order {k}")
        flags = np.zeros(e.G, np.int32)
        flags[e.order_kept(k)] = 1
        np.testing.assert_array_equal(layer.cum(k).cpu().numpy(), np.concatenate([[0], np.cumsum(flags)]))
        np.testing.assert_array_equal(layer.scales(k).cpu().numpy().view(np.uint32), e.order_scales(k).view(np.uint32),
                                      err_msg=f"scales, order {k}")
        np.testing.assert_array_equal(layer.codes(k).cpu().numpy(), e.packed(k), err_msg=f"codes, order {k}")
        if check_kernel_layout:
            np.testing.assert_array_equal(layer.kcodes(k).cpu().numpy(),
                                          kernel_layout_from_codes(e.order_codes(k), 2 if e.bits == 2 else (4 if e.bits <= 4 else 8)),
                                          err_msg=f"streaming layout, order {k}")
        w = layer.wcodes(k)
        if layer.desc.int8_copy:
            np.testing.assert_array_equal(w.cpu().numpy().view(np.int8), int8_copy_from_codes(e.order_codes(k)),
                                          err_msg=f"int8 copy, order {k}")
        else:
            assert w is None
    assert_block_tables_match(layer, e)


def int8_copy_from_codes(codes: np.ndarray) -> np.ndarray:
    """The int8 operand-layout copy (include/pipe.h) from int8 codes [rows, I]: [I_pad / 128, rows, 128], the 16-byte
    piece c of compacted row r stored as piece c ^ (r & 7)."""
    rows, I = codes.shape
    Ipad = (I + 127) // 128 * 128
    c = np.zeros((rows, Ipad), np.int8)
    c[:, :I] = codes
    pieces = c.reshape(rows, Ipad // 128, 8, 16)
    out = np.zeros_like(pieces)
    for a in range(8):          # rows with r & 7 == a
        for p in range(8):
            out[a::8, :, p ^ a, :] = pieces[a::8, :, p, :]
    return np.ascontiguousarray(out.transpose(1, 0, 2, 3)).reshape(Ipad // 128, rows, 128)


def expected_decode_table(kept_lists, G: int, g: int, row_limit: int, channel_limit: int = 512):
    """A decode-unit table: the same greedy cut with the row limit the layout states."""
    rows = np.zeros(G, np.int64)
    for kept in kept_lists:
        rows[np.asarray(kept)] += g
    bounds = [0]
    cur_rows, cur_groups = 0, 0
    for j in range(G):
        if cur_groups > 0 and (cur_rows + rows[j] > row_limit or (cur_groups + 1) * g > channel_limit):
            bounds.append(j)
            cur_rows, cur_groups = 0, 0
        cur_rows += int(rows[j])
        cur_groups += 1
    bounds.append(G)
    return np.array([len(bounds) - 1] + bounds, np.int32)


def expected_block_table(kept_lists, G: int, g: int, row_max: int = 256, channel_limit: int = 512):
    """The channel-block table of a cluster of orders as include/pipe.h defines it, from the kept-group lists: the
    row limit is the mean block size for the fewest possible blocks plus one group of every order (at most row_max);
    walk the groups from 0, close a block when the next group would take its stacked rows past the limit or its
    channels past channel_limit."""
    rows = np.zeros(G, np.int64)
    for kept in kept_lists:
        rows[np.asarray(kept)] += g
    R = int(rows.sum())
    half = len(kept_lists) * g // 2
    ne = max(-(-R // max(row_max - half, 1)), -(-(G * g) // channel_limit))
    if 1 <= ne <= B.EVEN_BLOCKS:
        row_limit = min(row_max, -(-R // ne) + half)
    else:
        n0 = max(-(-R // row_max), -(-(G * g) // channel_limit))
        row_limit = min(row_max, (-(-(-(-R // n0)) // 16)) * 16 + len(kept_lists) * g)
    bounds = [0]
    cur_rows, cur_groups = 0, 0
    for j in range(G):
        if cur_groups > 0 and (cur_rows + rows[j] > row_limit or (cur_groups + 1) * g > channel_limit):
            bounds.append(j)
            cur_rows, cur_groups = 0, 0
        cur_rows += int(rows[j])
        cur_groups += 1
    bounds.append(G)
    return np.array([len(bounds) - 1] + bounds, np.int32)


def expected_block_records(kept_lists, scale_lists, table, g):
    """The block records (pipe.h) of a channel-block table, from the definition: kept groups and scales of the cluster's
    orders (the ORACLE's), the table's boundaries."""
    n = int(table[0])
    nk = len(kept_lists)
    G = int(table[1 + n])
    # compacted row of every channel in every order, or -1
    crow = np.full((nk, G * g), -1, np.int64)
    for q, kept in enumerate(kept_lists):
        for i, j in enumerate(np.asarray(kept)):
            crow[q, j * g:(j + 1) * g] = i * g + np.arange(g)
    recs = np.zeros((n, B.BLOCK_RECORD_BYTES), np.uint8)
    for cb in range(n):
        j0, j1 = int(table[1 + cb]), int(table[2 + cb])
        c0, c1 = j0 * g, j1 * g
        hdr = np.zeros(32, np.int32)
        colmap = np.full(512, -1, np.int16)
        scale = np.zeros(256, np.float32)
        rb = 0
        for q in range(8):
            hdr[8 + q] = rb
            if q < nk:
                rows = crow[q, c0:c1]
                rows = rows[rows >= 0]
                hdr[16 + q] = int(np.sum(np.asarray(kept_lists[q]) < j0)) * g
                scale[rb:rb + len(rows)] = np.asarray(scale_lists[q])[rows]
                for cc in range((c1 - c0) // 8):
                    r = crow[q, c0 + 8 * cc]
                    if r >= 0:
                        colmap[8 * cc + q] = rb + r - hdr[16 + q]
                rb += len(rows)
        hdr[0], hdr[1], hdr[2], hdr[3] = c0, c1, nk, rb
        recs[cb, :128] = hdr.view(np.uint8)
        recs[cb, 128:128 + 1024] = colmap.view(np.uint8)
        recs[cb, 128 + 1024:] = scale.view(np.uint8)
    return recs


def assert_block_tables_match(layer: B.ExpandedLayer, e):
    """Every channel-block table of the blob against the definition evaluated on the ORACLE's kept lists."""
    lay = layer.layout
    M = layer.desc.num_branches
    split = [lay.branch_orders[m] for m in range(M)]
    begin = np.concatenate([[0], np.cumsum(split)])
    for m in range(M + 1):
        k0, k1 = (int(begin[m]), int(begin[m + 1])) if m < M else (0, e.K)
        table = layer.block_table(m)
        if (k1 - k0) > 8 or (k1 - k0) * e.g > 256:
            assert table is None
            continue
        want = expected_block_table([e.order_kept(k) for k in range(k0, k1)], e.G, e.g)
        got = table.cpu().numpy()
        assert want[0] <= lay.blk_cap[m]
        np.testing.assert_array_equal(got[:len(want)], want, err_msg=f"channel-block table {m}")
        assert want[0] <= lay.rec_cap[m]
        recs = layer.block_records(m).cpu().numpy()
        want_recs = expected_block_records([e.order_kept(k) for k in range(k0, k1)], [e.order_scales(k) for k in range(k0, k1)], want, e.g)
        np.testing.assert_array_equal(recs[:len(want_recs)], want_recs, err_msg=f"block records of table {m}")
        dtable = layer.decode_table(m)
        if dtable is not None:
            assert 16 <= lay.dec_limit[m] <= 256
            want = expected_decode_table([e.order_kept(k) for k in range(k0, k1)], e.G, e.g, lay.dec_limit[m])
            np.testing.assert_array_equal(dtable.cpu().numpy()[:len(want)], want, err_msg=f"decode-unit table {m}")


def gpu_quantize(x: np.ndarray, static_scale=None, xd=None):
    xd = torch.from_numpy(x).cuda() if xd is None else xd
    xq = torch.empty(xd.shape, dtype=torch.int8, device="cuda")
    sx = torch.zeros(1, dtype=torch.float32, device="cuda")
    ws = B.alloc_bytes(256)
    ss = None if static_scale is None else torch.tensor([static_scale], dtype=torch.float32, device="cuda")
    B.pipe_quantize_act(xd, xq, sx, ws, ss)
    torch.cuda.synchronize()
    return xq, sx


def gpu_linear(layer, xq, sx, bias=None, want_partials=True, kernel=B.KERNEL_AUTO):
    T = xq.shape[0]
    y = torch.full((T, layer.desc.out_features), float("nan"), dtype=torch.float32, device="cuda")
    part = torch.zeros((T, layer.layout.total_rows), dtype=torch.int32, device="cuda") if want_partials else None
    bd = None if bias is None else torch.from_numpy(bias).cuda()
    B.pipe_diag_select_kernel(kernel)
    try:
        B.pipe_expanded_linear(layer.desc, layer.blob, xq, sx, y, bd, part)
        torch.cuda.synchronize()
    finally:
        B.pipe_diag_select_kernel(B.KERNEL_AUTO)
    assert B.pipe_poll_status() == B.PIPE_OK
    return y.cpu().numpy(), (None if part is None else part.cpu().numpy())


def gpu_ensemble(layer, xq_m, sx_m, bias=None, sum_branches=False, want_partials=True, kernel=B.KERNEL_AUTO):
    M = layer.desc.num_branches
    T = xq_m[0].shape[0]
    O = layer.desc.out_features
    n_out = 1 if sum_branches else M
    ys = [torch.full((T, O), float("nan"), dtype=torch.float32, device="cuda") for _ in range(n_out)]
    part = torch.zeros((T, layer.layout.total_rows), dtype=torch.int32, device="cuda") if want_partials else None
    bd = None if bias is None else torch.from_numpy(bias).cuda()
    B.pipe_diag_select_kernel(kernel)
    try:
        B.pipe_ensemble_forward(layer.desc, layer.blob, xq_m, sx_m, ys, bd, sum_branches, part)
        torch.cuda.synchronize()
    finally:
        B.pipe_diag_select_kernel(B.KERNEL_AUTO)
    assert B.pipe_poll_status() == B.PIPE_OK
    return [y.cpu().numpy() for y in ys], (None if part is None else part.cpu().numpy())


def gpu_ensemble_q8(layer, xq_m, sx_m, out_scales, bias=None, relu=True, want_partials=True, kernel=B.KERNEL_AUTO,
                    pitch_extra=0):
    """Inner layer of the M predictors through pipe_ensemble_forward_q8; out_scales: M floats.  Returns the M
    int8 outputs (numpy) and the partials.  pitch_extra > 0 gives the outputs a row pitch of O + pitch_extra."""
    M = layer.desc.num_branches
    T = xq_m[0].shape[0]
    O = layer.desc.out_features
    bufs = [torch.full((T, O + pitch_extra), 99, dtype=torch.int8, device="cuda") for _ in range(M)]
    yq = [b[:, :O] for b in bufs]
    so = [torch.tensor([s], dtype=torch.float32, device="cuda") for s in out_scales]
    part = torch.zeros((T, layer.layout.total_rows), dtype=torch.int32, device="cuda") if want_partials else None
    bd = None if bias is None else torch.from_numpy(bias).cuda()
    B.pipe_diag_select_kernel(kernel)
    try:
        B.pipe_ensemble_forward_q8(layer.desc, layer.blob, xq_m, sx_m, so, yq, bd, relu, part)
        torch.cuda.synchronize()
    finally:
        B.pipe_diag_select_kernel(B.KERNEL_AUTO)
    if pitch_extra:
        for b in bufs:
            assert (b[:, O:] == 99).all(), "bytes beyond the row were written"
    return [y.cpu().numpy() for y in yq], (None if part is None else part.cpu().numpy())


def assert_outputs_close(y_gpu: np.ndarray, f, what=""):
    """f: oracle Forward (y, y64, yabs).  The stated tolerance, element-wise, against the binary64 sum."""
    err = np.abs(y_gpu.astype(np.float64) - f.y64)
    bound = REL_TOL * f.yabs + 1e-30
    bad = err > bound
    assert not bad.any(), f"{what}: {bad.sum()} outputs beyond 1e-5 relative; worst {np.max(err / (f.yabs + 1e-30)):.3e}"
