"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU).

Each test names the passage it checks.  None of them re-types the oracle's own formula:
they use closed forms, invariants, NumPy library routines on special cases, the paper's
printed ensemble splits and budgets, and an exact-rational brute force (tests/exact.py).
"""
import os
from fractions import Fraction

import numpy as np
import pytest

from tests import exact

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand_w(rng, O, I, heavy=False):
    W = (rng.standard_t(4, size=(O, I)) if heavy else rng.standard_normal((O, I))) * 0.02
    W *= np.exp(rng.uniform(np.log(0.5), np.log(2.0), size=(O, 1)))
    return W.astype(np.float32)


def _recon64(e, upto=None):
    """sum_k s_k q_k in binary64 from the EMITTED codes and scales, dense [O, I]."""
    out = np.zeros((e.O, e.I), np.float64)
    for k in range(e.K if upto is None else upto):
        ch = e.order_channels(k)
        out[ch] += e.order_scales(k).astype(np.float64)[:, None] * e.order_codes(k).astype(np.float64)
    return out


# ----------------------------------------------------------------------------------------------
# Eq. 1 / Sec. 3: code range of a symmetric b-bit quantizer; ternary is {-1, 0, +1}.
@pytest.mark.parametrize("bits", [8, 4, 2])
def test_code_range_and_scale_definition(oracle, bits):
    rng = np.random.default_rng(10 + bits)
    W = _rand_w(rng, 32, 40, heavy=True)
    e = oracle.expand(W, bits, 3, 8, 4)
    qmax = 2 ** (bits - 1) - 1
    assert e.codes.min() >= -qmax and e.codes.max() <= qmax
    # first-order scale: row absmax / qmax, and the absmax element maps to +-qmax
    s1 = e.order_scales(0)
    np.testing.assert_array_equal(s1, (np.abs(W).max(axis=1) / np.float32(qmax)).astype(np.float32))
    assert (np.abs(e.order_codes(0)).max(axis=1) == qmax).all()
    if bits == 2:
        assert set(np.unique(e.codes)) <= {-1, 0, 1}


# ----------------------------------------------------------------------------------------------
# Sec. 3.1: "the support of the quantization error space is smaller than one quantization
# step": after order k every kept row's residual is at most half a step s_k (one binary32
# rounding of slack), and the tracked residual equals W - sum s_k q_k.
@pytest.mark.parametrize("bits,K", [(8, 3), (4, 4), (2, 6)])
def test_residual_within_half_step_and_tracks_reconstruction(oracle, bits, K):
    rng = np.random.default_rng(20 + bits)
    W = _rand_w(rng, 24, 64)
    e = oracle.expand(W, bits, K, 8, 3)  # gamma = 1
    for k in range(K):
        nxt = e.absmax[k + 1] if k + 1 < K else np.abs(e.residual).max(axis=1)
        ch = e.order_channels(k)
        half = e.order_scales(k).astype(np.float64) / 2 * (1 + 2.0 ** -22)
        assert (nxt[ch].astype(np.float64) <= half).all(), f"order {k}"
    err = W.astype(np.float64) - _recon64(e)
    # each order's tracked residual carries at most one rounding of a value <= s_k/2
    slack = sum(e.order_scales(k).astype(np.float64) for k in range(K)) * 2.0 ** -24
    assert (np.abs(err - e.residual.astype(np.float64)) <= slack[:, None]).all()


# ----------------------------------------------------------------------------------------------
# Sec. 3.1: "the error decreases by a factor larger than 2^b with each expansion term".
# With codes in [-qmax, qmax] the guaranteed factor per order is 2*qmax = 2^b - 2
# (for b = 2 the scale halves); measured on the emitted scales.
@pytest.mark.parametrize("bits", [8, 4, 2])
def test_scale_contraction_per_order(oracle, bits):
    rng = np.random.default_rng(30 + bits)
    W = _rand_w(rng, 16, 128, heavy=True)
    K = 4
    e = oracle.expand(W, bits, K, 8, 2)
    qmax = 2 ** (bits - 1) - 1
    for k in range(K - 1):
        s0 = e.order_scales(k).astype(np.float64)
        s1 = e.order_scales(k + 1).astype(np.float64)
        assert (s1 <= s0 / (2 * qmax) * (1 + 1e-6)).all()
    # and the typical factor is of the order the paper states (within a factor 2 of 2^b)
    ratio = np.median(e.order_scales(0).astype(np.float64) / e.order_scales(1).astype(np.float64))
    assert 2 * qmax * (1 - 1e-6) <= ratio <= 2 ** (bits + 1)


# ----------------------------------------------------------------------------------------------
# Lemma B.1 (Eq. 7): |w - sum_{k<=K} w^(k)| <= (1/(2^(b-1)-1))^(K-1) * lambda_i / 2, lambda the
# row's FIRST-order scale (reading: with the K-th order scale the printed inequality fails
# for K >= 2).  Evaluated from the emitted codes/scales, for every K; and non-increasing in K.
@pytest.mark.parametrize("bits", [8, 4, 2])
def test_lemma_b1_exponential_decrease(oracle, bits):
    rng = np.random.default_rng(40 + bits)
    W = _rand_w(rng, 16, 96)
    qmax = 2 ** (bits - 1) - 1
    Kmax = 5
    e = oracle.expand(W, bits, Kmax, 8, 2)
    s1 = e.order_scales(0).astype(np.float64)
    prev = None
    for K in range(1, Kmax + 1):
        err = np.abs(W.astype(np.float64) - _recon64(e, K)).max(axis=1)
        bound = (1.0 / qmax) ** (K - 1) * s1 / 2
        assert (err <= bound * (1 + 1e-6) + 1e-12).all(), f"K={K}"
        if prev is not None:
            assert (err <= prev * (1 + 1e-9) + 1e-12).all()
        prev = err
    # the reading matters: lambda = s_K would make the printed bound false at K = 2 (b > 2)
    if bits > 2:
        err2 = np.abs(W.astype(np.float64) - _recon64(e, 2)).max(axis=1)
        wrong = (1.0 / qmax) * e.order_scales(1).astype(np.float64) / 2
        assert (err2 > wrong).any()


# ----------------------------------------------------------------------------------------------
# Exact recovery of already-representable weights: W = s*Q with s a power of two per row and
# max|Q| = qmax gives back (Q, s) exactly and every higher order is zero; a two-term sum
# s*Q1 + s'*Q2 is separated exactly into orders 1 and 2.
@pytest.mark.parametrize("bits", [8, 4, 2])
def test_exact_recovery_of_representable_weights(oracle, bits):
    rng = np.random.default_rng(50 + bits)
    qmax = 2 ** (bits - 1) - 1
    O, I = 16, 48
    Q1 = rng.integers(-qmax, qmax + 1, size=(O, I))
    Q1[:, 0] = qmax * (rng.integers(0, 2, size=O) * 2 - 1)
    s = 2.0 ** rng.integers(-12, -3, size=O)
    W = (s[:, None] * Q1).astype(np.float32)
    e = oracle.expand(W, bits, 3, 8, 2)
    np.testing.assert_array_equal(e.order_codes(0), Q1)
    np.testing.assert_array_equal(e.order_scales(0), s.astype(np.float32))
    assert not e.order_codes(1).any() and not e.order_scales(1).any()
    assert not e.order_codes(2).any() and not e.residual.any()

    if bits > 2:
        p = bits + 1  # s' = s / 2^p  =>  |s' Q2| <= s*qmax/2^p < s/2
        Q2 = rng.integers(-qmax, qmax + 1, size=(O, I))
        Q1[:, 1] = 0
        W = (s[:, None] * Q1).astype(np.float32)
        Q2[np.abs(Q1) == qmax] = 0        # keep the row absmax at s*qmax
        Q2[:, 1] = qmax                   # and order 2's absmax at s'*qmax
        s2 = s / 2.0 ** p
        W2 = (s[:, None] * Q1 + s2[:, None] * Q2).astype(np.float32)
        assert (W2.astype(np.float64) == s[:, None] * Q1 + s2[:, None] * Q2).all()  # exact in binary32
        e2 = oracle.expand(W2, bits, 3, 8, 2)
        np.testing.assert_array_equal(e2.order_codes(0), Q1)
        np.testing.assert_array_equal(e2.order_codes(1), Q2)
        np.testing.assert_array_equal(e2.order_scales(1), s2.astype(np.float32))
        assert not e2.order_codes(2).any() and not e2.residual.any()


# ----------------------------------------------------------------------------------------------
# gamma = 1 and M = 1 is the plain (unmasked) expansion of Eq. 3: every order keeps all
# groups, and its codes are those of a direct NumPy evaluation of Q on W - sum of the
# emitted lower orders (binary64 difference, exact here, rounded once to binary32).
def test_gamma_one_is_plain_expansion(oracle):
    rng = np.random.default_rng(60)
    W = _rand_w(rng, 32, 40)
    bits, K, g = 4, 3, 8
    e = oracle.expand(W, bits, K, g, 32 // g)
    qmax = 7
    for k in range(K):
        np.testing.assert_array_equal(e.order_kept(k), np.arange(4))
        r = (W.astype(np.float64) - _recon64(e, k)).astype(np.float32)
        s = (np.abs(r).max(axis=1) / np.float32(qmax)).astype(np.float32)
        q = np.clip(np.rint(r / s[:, None]), -qmax, qmax).astype(np.int8)
        np.testing.assert_array_equal(e.order_scales(k), s)
        np.testing.assert_array_equal(e.order_codes(k), q)


# ----------------------------------------------------------------------------------------------
# Structured mask (Sec. 3.1, masked equation; Sec. 4.1 "sparsity is applied to the neurons"):
# selection invariants of the reading "keep the n groups with the largest residual max-abs".
def test_selection_invariants(oracle):
    rng = np.random.default_rng(70)
    O, I, g, n_keep, K = 64, 32, 8, 3, 4
    W = _rand_w(rng, O, I, heavy=True)
    e = oracle.expand(W, 4, K, g, n_keep)
    G = O // g
    assert int(e.kept_count[0]) == G
    seen = set()
    for k in range(1, K):
        kept = e.order_kept(k)
        assert len(kept) == n_keep and (np.diff(kept) > 0).all() and kept.min() >= 0 and kept.max() < G
        score = e.absmax[k].reshape(G, g).max(axis=1)
        pruned = np.setdiff1d(np.arange(G), kept)
        assert score[kept].min() >= score[pruned].max()
        # pruned rows: residual (hence absmax) carries over unchanged to the next order
        if k + 1 < K:
            rows = (pruned[:, None] * g + np.arange(g)).reshape(-1)
            np.testing.assert_array_equal(e.absmax[k + 1][rows], e.absmax[k][rows])
        seen.add(tuple(kept))
    assert len(seen) > 1  # different orders keep different groups on this input
    # effective rows = O * (1 + (K-1) * gamma)
    assert e.R_total == O + (K - 1) * n_keep * g


def test_selection_ties_go_to_lower_index(oracle):
    a = np.zeros(48, np.float32)
    a[[0, 9, 17, 30, 41]] = [3.0, 5.0, 3.0, 3.0, 1.0]      # groups of 8: scores 3,5,3,3,0,1
    np.testing.assert_array_equal(oracle.select_groups(a, 8, 3), [0, 1, 2])
    np.testing.assert_array_equal(oracle.select_groups(a, 8, 1), [1])
    np.testing.assert_array_equal(oracle.select_groups(a, 8, 5), [0, 1, 2, 3, 5])
    np.testing.assert_array_equal(oracle.select_groups(np.ones(32, np.float32), 4, 3), [0, 1, 2])


def test_keep_groups_from_gamma(oracle):
    # every configuration of the benchmark has an integral gamma*G
    assert oracle.keep_groups(32, 0.25) == 8 and oracle.keep_groups(384, 0.5) == 192
    assert oracle.keep_groups(1376, 0.5) == 688 and oracle.keep_groups(512, 0.25) == 128
    assert oracle.keep_groups(10, 0.33) == 4 and oracle.keep_groups(10, 0.3) == 3
    assert oracle.keep_groups(10, 0.0) == 1 and oracle.keep_groups(10, 1.0) == 10 and oracle.keep_groups(7, 2.0) == 7
    with open(os.path.join(GOLDEN, "budgets.txt")) as f:
        for line in f:
            line = line.split("#")[0].split()
            if not line:
                continue
            K, gamma, cost = int(line[0]), float(line[1]), float(line[2])
            G = 56
            rows = G + (K - 1) * oracle.keep_groups(G, gamma)
            assert abs(rows / G - cost) < 1e-9


# ----------------------------------------------------------------------------------------------
# Eq. 9 special case: K = 1, b = 8, one cluster is a textbook int8 x int8 -> int32 matmul and a
# row/column scaling; compare with NumPy's integer matmul and a binary64 scaling.
def test_single_order_int8_reduces_to_integer_matmul(oracle):
    rng = np.random.default_rng(80)
    O, I, T = 24, 80, 12
    W = _rand_w(rng, O, I)
    x = rng.standard_normal((T, I)).astype(np.float32)
    e = oracle.expand(W, 8, 1, 8, 3)
    xq, sx = oracle.quantize_act(x)
    f = oracle.forward(e, xq, sx)
    acc = xq.astype(np.int64) @ e.order_codes(0).astype(np.int64).T
    np.testing.assert_array_equal(f.partials, acc)
    ref = acc * e.order_scales(0).astype(np.float64)[None, :] * float(sx)
    np.testing.assert_allclose(f.y, ref, rtol=3e-7, atol=0)
    np.testing.assert_allclose(f.y64, ref, rtol=1e-14)
    # and the whole thing approximates the fp32 layer to quantization accuracy
    exact_y = x.astype(np.float64) @ W.astype(np.float64).T
    assert np.abs(f.y - exact_y).max() < 0.05 * np.abs(exact_y).max()


def test_activation_quantizer(oracle):
    rng = np.random.default_rng(81)
    x = rng.standard_normal((7, 33)).astype(np.float32) * 3
    xq, sx = oracle.quantize_act(x)
    assert sx == np.float32(np.abs(x).max() / np.float32(127))
    assert np.abs(xq).max() == 127 and (np.abs(xq.astype(np.float64) * float(sx) - x) <= float(sx) / 2 * (1 + 1e-6)).all()
    # ties to even at exactly representable half-steps
    xs = np.array([[0.5, 1.5, 2.5, -0.5, -1.5, 127.0, 3.5, -2.5]], np.float32)
    q, s = oracle.quantize_act(xs)
    assert s == np.float32(1.0)
    np.testing.assert_array_equal(q, [[0, 2, 2, 0, -2, 127, 4, -2]])
    # static scale clamps
    q, s = oracle.quantize_act(np.array([[300.0, -300.0, 1.0]], np.float32), static_scale=1.0)
    np.testing.assert_array_equal(q, [[127, -127, 1]])
    q, s = oracle.quantize_act(np.zeros((2, 5), np.float32))
    assert s == 0 and not q.any()
    with pytest.raises(oracle.OracleError):
        oracle.quantize_act(np.array([[np.nan, 1.0]], np.float32))


def test_weight_ties_round_to_even(oracle):
    # row absmax 7 with b = 4 gives s = 1: codes are rne of the values themselves
    W = np.array([[7.0, 0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 6.5]], np.float32)
    e = oracle.expand(W, 4, 1, 1, 1)
    np.testing.assert_array_equal(e.order_codes(0), [[7, 0, 2, 2, 0, -2, -2, 6]])


# ----------------------------------------------------------------------------------------------
# Sec. 3.2 / Fig. 2 / Appendix B: clusters of successive orders, bias in predictor 1 only,
# sum after the layer; and the printed splits.
def test_printed_ensemble_splits(oracle):
    with open(os.path.join(GOLDEN, "ensemble_splits.txt")) as f:
        n = 0
        for line in f:
            line = line.split("#")[0].split()
            if not line:
                continue
            K, M, split = int(line[0]), int(line[1]), [int(v) for v in line[2].split(",")]
            np.testing.assert_array_equal(oracle.balanced_split(K, M), split)
            n += 1
    assert n == 5


def test_ensemble_identities(oracle):
    rng = np.random.default_rng(90)
    O, I, T, K, g, n_keep = 32, 48, 9, 4, 8, 2
    W = _rand_w(rng, O, I)
    bias = rng.standard_normal(O).astype(np.float32)
    e = oracle.expand(W, 4, K, g, n_keep)
    x = rng.standard_normal((T, I)).astype(np.float32)
    xq, sx = oracle.quantize_act(x)
    full = oracle.forward(e, xq, sx, bias=bias)
    # shared input, split [2,2], summed: integer partials identical, fp32 sum equal up to re-association
    xs = np.stack([xq, xq])
    y_sum, p_sum = oracle.ensemble(e, xs, [sx, sx], [2, 2], bias=bias, sum_branches=True)
    np.testing.assert_array_equal(p_sum, full.partials)
    assert (np.abs(y_sum - full.y64) <= 1e-6 * full.yabs + 1e-30).all()
    # M = 1 is exactly the expanded layer
    y1, p1 = oracle.ensemble(e, xq[None], [sx], [K], bias=bias, sum_branches=True)
    np.testing.assert_array_equal(y1, full.y)
    # per-branch outputs: bias only in branch 1; branch m only sees its own orders and its own input
    x2 = rng.standard_normal((T, I)).astype(np.float32)
    xq2, sx2 = oracle.quantize_act(x2)
    ym, pm = oracle.ensemble(e, np.stack([xq, xq2]), [sx, sx2], [2, 2], bias=bias)
    b0 = oracle.forward(e, xq, sx, 0, 2, bias=bias)
    b1 = oracle.forward(e, xq2, sx2, 2, 4)
    np.testing.assert_array_equal(ym[0], b0.y)
    np.testing.assert_array_equal(ym[1], b1.y)
    nb = oracle.forward(e, xq, sx, 0, 2)
    np.testing.assert_allclose(b0.y64 - nb.y64, np.broadcast_to(bias.astype(np.float64), (T, O)), atol=1e-12)
    # the expanded layer approaches the fp32 layer as orders are added (dense expansion)
    ed = oracle.expand(W, 4, K, g, O // g)
    exact_y = (xq.astype(np.float64) * float(sx)) @ W.astype(np.float64).T
    errs = [np.abs(oracle.forward(ed, xq, sx, 0, k).y64 - exact_y).max() for k in range(1, K + 1)]
    assert all(errs[i + 1] < errs[i] / 4 for i in range(K - 1))


def test_pruned_rows_contribute_nothing(oracle):
    rng = np.random.default_rng(91)
    O, I, T, g = 32, 16, 5, 8
    W = _rand_w(rng, O, I)
    e = oracle.expand(W, 4, 2, g, 1)
    xq, sx = oracle.quantize_act(rng.standard_normal((T, I)).astype(np.float32))
    y1 = oracle.forward(e, xq, sx, 0, 1).y
    y2 = oracle.forward(e, xq, sx, 0, 2).y
    kept_rows = e.order_channels(1)
    pruned = np.setdiff1d(np.arange(O), kept_rows)
    np.testing.assert_array_equal(y1[:, pruned], y2[:, pruned])
    assert (y1[:, kept_rows] != y2[:, kept_rows]).any()


# ----------------------------------------------------------------------------------------------
# Storage format of the packed codes.
def test_packing_bit_order(oracle):
    c = np.array([[1, -1, 7, -7, 0, 3, -8 + 1, 2]], np.int8)
    p4 = oracle.pack(c, 4)
    np.testing.assert_array_equal(p4, [[0xF1, 0x97, 0x30, 0x29]])
    t = np.array([[1, 0, -1, 1, -1, -1, 0, 0, 1]], np.int8)
    p2 = oracle.pack(t, 2)
    np.testing.assert_array_equal(p2, [[0b01110001, 0b00001111, 0b00000001]])
    np.testing.assert_array_equal(oracle.pack(c, 8).view(np.int8), c)


# ----------------------------------------------------------------------------------------------
# Brute force on tiny inputs, every stage, exact rational arithmetic (tests/exact.py).
@pytest.mark.parametrize("bits,K,g,n_keep,seed", [(8, 2, 2, 2, 0), (4, 3, 2, 1, 1), (2, 4, 2, 2, 2), (4, 4, 4, 1, 3),
                                                  (2, 3, 1, 3, 4), (8, 3, 2, 3, 5)])
def test_brute_force_tiny(oracle, bits, K, g, n_keep, seed):
    rng = np.random.default_rng(100 + seed)
    O, I, T = 8, 8, 3
    W = (rng.standard_t(3, size=(O, I)) * 0.05).astype(np.float32)
    W[1] = 0.0                       # an all-zero row
    W[2, :] = W[3, :]                # equal rows -> equal scores
    x = rng.standard_normal((T, I)).astype(np.float32)
    bias = rng.standard_normal(O).astype(np.float32)
    e = oracle.expand(W, bits, K, g, n_keep)
    codes, scales, kept, resid = exact.expand_exact(W, bits, K, g, n_keep)
    for k in range(K):
        np.testing.assert_array_equal(e.order_kept(k), kept[k])
        ch = e.order_channels(k)
        for n, o in enumerate(ch):
            assert list(e.order_codes(k)[n]) == codes[k][o], (k, o)
            assert Fraction(float(e.order_scales(k)[n])) == scales[k][o], (k, o)
    for o in range(O):
        assert [Fraction(float(v)) for v in e.residual[o]] == resid[o]
    xq, sx = oracle.quantize_act(x)
    xq_e, sx_e = exact.quantize_act_exact(x)
    np.testing.assert_array_equal(xq, xq_e)
    assert Fraction(float(sx)) == sx_e
    k_split = max(1, K // 2)
    for (k0, k1, b) in [(0, K, bias), (0, k_split, None), (k_split, K, None)]:
        if k0 >= k1:
            continue
        f = oracle.forward(e, xq, sx, k0, k1, bias=b)
        y_e, part_e = exact.forward_exact(codes, scales, xq_e, sx_e, k0, k1, O, bias=b)
        for t in range(T):
            assert [Fraction(float(v)) for v in f.y[t]] == y_e[t]
        for k in range(k0, k1):
            ch = e.order_channels(k)
            for n, o in enumerate(ch):
                assert list(f.partials[:, e.row_off(k) + n]) == part_e[(k, o)]


def test_nonfinite_weights_are_rejected(oracle):
    W = np.ones((8, 8), np.float32)
    W[3, 4] = np.inf
    with pytest.raises(oracle.OracleError) as ei:
        oracle.expand(W, 4, 2, 8, 1)
    assert ei.value.code == oracle.ERR_NONFINITE


def test_accumulator_overflow_is_detected(oracle):
    # 127 * 127 * I exceeds int32 for I > 133143
    I = 133200
    W = np.full((1, I), 1.0, np.float32)
    e = oracle.expand(W, 8, 1, 1, 1)
    xq = np.full((1, I), 127, np.int8)
    with pytest.raises(oracle.OracleError) as ei:
        oracle.forward(e, xq, 1.0)
    assert ei.value.code == oracle.ERR_ACC_OVERFLOW


def test_requantized_branch_is_the_composition_and_a_two_layer_chain_closes(oracle):
    """Sec. 3.2 / App. B: a branch of an inner layer hands sigma(its cluster's output), quantized by the next
    layer's Q, to the same branch of the next layer.  The helper is the composition of the pinned pieces, and
    with every order in one branch and codes that reproduce the weights exactly the two-layer chain equals the
    plain integer network computed with NumPy."""
    rng = np.random.default_rng(3)
    O1, I1, O2, T = 24, 16, 8, 9
    # weights that one 8-bit order represents exactly: s * integers with a full-range entry per row
    q1 = rng.integers(-127, 128, size=(O1, I1)); q1[:, 0] = 127
    q2 = rng.integers(-127, 128, size=(O2, O1)); q2[:, 0] = -127
    s1, s2 = np.float32(2.0 ** -9), np.float32(2.0 ** -7)
    W1, W2 = (q1 * s1).astype(np.float32), (q2 * s2).astype(np.float32)
    e1, e2 = oracle.expand(W1, 8, 1, 8, O1 // 8), oracle.expand(W2, 8, 1, 8, O2 // 8)
    xq = rng.integers(-127, 128, size=(T, I1)).astype(np.int8)
    sx, s_mid = np.float32(2.0 ** -6), np.float32(2.0 ** -3)
    hq = oracle.forward_requantized(e1, xq, sx, float(s_mid))
    # composition
    y1 = oracle.forward(e1, xq, sx).y
    want, _ = oracle.quantize_act(np.maximum(y1, 0), static_scale=float(s_mid))
    np.testing.assert_array_equal(hq, want)
    # plain integer network: every product below is a power-of-two multiple of an integer, exact in binary64
    a1 = (xq.astype(np.int64) @ q1.T).astype(np.float64) * float(s1) * float(sx)
    h_int = np.clip(np.rint(np.maximum(a1, 0) / float(s_mid)), -127, 127).astype(np.int64)
    np.testing.assert_array_equal(hq.astype(np.int64), h_int)
    y2 = oracle.forward(e2, hq, s_mid).y
    np.testing.assert_array_equal(y2.astype(np.float64), (h_int @ q2.T).astype(np.float64) * float(s2) * float(s_mid))
