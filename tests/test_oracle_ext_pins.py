"""Pins of the oracle's variants beside the main setting (oracle/pipe_oracle_ext.c; no GPU): other weight
bit-widths (Sec. 4.2), narrower and asymmetric activations (Sec. 4.3), the second group score and the
unstructured mask (Sec. 3.1), the activation functions of Sec. 3.2.  As for the main pins, nothing here re-types
the oracle's own code: invariants, closed forms, NumPy / math library routines, exact-rational brute force.
"""
import math
from fractions import Fraction

import numpy as np
import pytest

from tests import exact


def _rand_w(rng, O, I):
    W = rng.standard_normal((O, I)) * 0.02 * np.exp(rng.uniform(np.log(0.5), np.log(2.0), size=(O, 1)))
    return W.astype(np.float32)


def _recon64(e):
    out = np.zeros((e.O, e.I), np.float64)
    for k in range(e.K):
        ch = e.order_channels(k)
        out[ch] += e.order_scales(k).astype(np.float64)[:, None] * e.order_codes(k).astype(np.float64)
    return out


# ---------------------------------------------------------------------------------------------------
# Sec. 4.2: the method at int3 and int6.  The same invariants that pin int8 / int4 / ternary.
@pytest.mark.parametrize("bits", [3, 6])
def test_other_bit_widths_keep_the_invariants(oracle, bits):
    rng = np.random.default_rng(bits)
    W = _rand_w(rng, 24, 50)
    qmax = 2 ** (bits - 1) - 1
    for K in (1, 2, 4):
        e = oracle.expand_ex(W, bits, K, 4, 6)
        assert np.abs(e.codes).max() == qmax                       # the row maximum hits the end of the range
        s1 = e.order_scales(0).astype(np.float64)
        np.testing.assert_array_equal(e.order_scales(0), (np.abs(W).max(axis=1) / np.float32(qmax)).astype(np.float32))
        err = np.abs(W.astype(np.float64) - _recon64(e)).max(axis=1)
        # Lemma B.1 with the first-order scale: error <= (1/qmax)^(K-1) * s_1 / 2, and the residual the oracle tracks
        # is the true one
        assert (err <= (1.0 / qmax) ** (K - 1) * s1 / 2 * (1 + 1e-6)).all()
        np.testing.assert_allclose(e.residual, W.astype(np.float64) - _recon64(e), rtol=0, atol=1e-9)
        # round-to-nearest leaves every last-order row within half a step
        last = e.order_scales(K - 1).astype(np.float64)
        assert (np.abs(e.residual).max(axis=1) <= last / 2 * (1 + 2.0 ** -20)).all()


@pytest.mark.parametrize("bits", [3, 6])
def test_other_bit_widths_recover_representable_weights(oracle, bits):
    rng = np.random.default_rng(10 + bits)
    qmax = 2 ** (bits - 1) - 1
    Q = rng.integers(-qmax, qmax + 1, size=(8, 33))
    Q[:, 0] = qmax * np.where(rng.integers(0, 2, 8) == 1, 1, -1)
    s = 2.0 ** rng.integers(-9, -3, size=8)
    W = (s[:, None] * Q).astype(np.float32)
    e = oracle.expand_ex(W, bits, 3, 4, 2)
    np.testing.assert_array_equal(e.order_codes(0), Q)
    np.testing.assert_array_equal(e.order_scales(0), s.astype(np.float32))
    assert not e.order_codes(1).any() and not e.order_scales(1).any() and not e.residual.any()


@pytest.mark.parametrize("bits", [8, 4, 2])
def test_the_general_expansion_reduces_to_the_pinned_one(oracle, bits):
    rng = np.random.default_rng(20 + bits)
    W = _rand_w(rng, 32, 40)
    a, b = oracle.expand(W, bits, 3, 4, 3), oracle.expand_ex(W, bits, 3, 4, 3)
    np.testing.assert_array_equal(a.codes, b.codes)
    np.testing.assert_array_equal(a.scales.view(np.uint32), b.scales.view(np.uint32))
    np.testing.assert_array_equal(a.kept, b.kept)
    np.testing.assert_array_equal(a.residual.view(np.uint32), b.residual.view(np.uint32))


def test_three_bit_codes_travel_in_nibbles_and_six_bit_codes_in_bytes(oracle):
    codes = np.array([[3, -3, 1, -1, 0, 2]], np.int8)
    np.testing.assert_array_equal(oracle.pack_ex(codes, 3), np.array([[0xD3, 0xF1, 0x20]], np.uint8))
    np.testing.assert_array_equal(oracle.pack_ex(np.array([[31, -31, -1]], np.int8), 6), np.array([[31, 225, 255]], np.uint8))
    assert [oracle.container_bits(b) for b in (2, 3, 4, 6, 8)] == [2, 4, 4, 8, 8]


# ---------------------------------------------------------------------------------------------------
# Sec. 4.3: A6 and A4 activations (symmetric).
@pytest.mark.parametrize("act_bits", [4, 6, 8])
def test_narrow_symmetric_activations(oracle, act_bits):
    qx = 2 ** (act_bits - 1) - 1
    rng = np.random.default_rng(act_bits)
    x = rng.standard_normal((6, 20)).astype(np.float32)
    xq, sx, zp = oracle.quantize_act_ex(x, act_bits)
    assert zp == 0 and np.abs(xq).max() == qx
    assert sx == np.float32(np.abs(x).max()) / np.float32(qx)
    # exact-rational restatement of Eq. 1
    want = [[max(-qx, min(qx, exact.rne_int(exact.f32(exact.frac(v) / exact.frac(sx))))) for v in row] for row in x]
    np.testing.assert_array_equal(xq, np.array(want))
    # ties go to the even code: with a power-of-two step every half-integer quotient is exact
    step = 2.0 ** -3
    ties = np.array([[(k + 0.5) * step for k in range(-qx, qx)]], np.float32)
    got = oracle.quantize_act_ex(ties, act_bits, static_scale=step)[0][0]
    for k, c in zip(range(-qx, qx), got):
        assert c in (k, k + 1) and c % 2 == 0
    if act_bits == 8:   # the int8 case is the pinned quantizer
        a, b = oracle.quantize_act(x)
        np.testing.assert_array_equal(a, xq)
        assert b == sx


# Sec. 4.3 (parallelized comparison): asymmetric activation quantization.
@pytest.mark.parametrize("act_bits", [4, 8])
def test_asymmetric_activations(oracle, act_bits):
    half = 2 ** (act_bits - 1)
    rng = np.random.default_rng(40 + act_bits)
    x = np.maximum(rng.standard_normal((7, 30)), -0.3).astype(np.float32) * 2   # skewed: most of the mass is positive
    c, lam, z = oracle.quantize_act_ex(x, act_bits, asymmetric=True)
    assert c.min() >= -half and c.max() <= half - 1
    assert c.min() == -half and c.max() == half - 1      # both ends of the range are used
    assert -half <= z <= half - 1
    # zero is represented exactly, and the reconstruction is within half a step everywhere
    zero = oracle.quantize_act_ex(np.concatenate([x.reshape(-1), [0.0]]).astype(np.float32)[None, :], act_bits, asymmetric=True,
                                  static_range=(float(x.min()), float(x.max())))[0][0, -1]
    assert zero == z
    recon = float(lam) * (c.astype(np.float64) - z)
    assert np.abs(recon - x).max() <= 0.5 * float(lam) * (1 + 1e-5) + float(lam) * 0.5   # z itself is rounded: one more half step
    # the step is the range over the number of levels
    assert lam == (np.float32(max(x.max(), 0)) - np.float32(min(x.min(), 0))) / np.float32(2 * half - 1)
    # a non-negative tensor (post-ReLU) maps its zero to the lowest code
    relu = np.maximum(x, 0)
    c2, lam2, z2 = oracle.quantize_act_ex(relu, act_bits, asymmetric=True)
    assert z2 == -half and c2.min() == -half


def test_zero_point_folds_into_a_row_sum(oracle):
    rng = np.random.default_rng(5)
    W = _rand_w(rng, 16, 24)
    e = oracle.expand_ex(W, 4, 3, 4, 2)
    x = np.maximum(rng.standard_normal((5, 24)), -0.2).astype(np.float32)
    c, lam, z = oracle.quantize_act_ex(x, 8, asymmetric=True)
    f, rowsum = oracle.forward_zp(e, c, lam, z)
    # NumPy integer matmul on the shifted codes, order by order
    for k in range(e.K):
        q = e.order_codes(k).astype(np.int64)
        lo = e.row_off(k)
        want = (c.astype(np.int64) - z) @ q.T
        np.testing.assert_array_equal(f.partials[:, lo:lo + e.rows(k)], want)
        np.testing.assert_array_equal(rowsum[lo:lo + e.rows(k)], q.sum(axis=1))
        # the identity an implementation uses
        np.testing.assert_array_equal(want, c.astype(np.int64) @ q.T - z * q.sum(axis=1)[None, :])
    # zero point 0 is the symmetric forward
    cs, ls = oracle.quantize_act(x)
    a = oracle.forward(e, cs, ls)
    b, _ = oracle.forward_zp(e, cs, ls, 0)
    np.testing.assert_array_equal(a.y.view(np.uint32), b.y.view(np.uint32))
    np.testing.assert_array_equal(a.partials, b.partials)
    # and the result approximates the float layer about as well as the symmetric one does
    dense = x.astype(np.float64) @ (W.astype(np.float64) - e.residual.astype(np.float64)).T
    assert np.abs(f.y64 - dense).max() <= 1.2 * float(lam) * np.abs(W).sum(axis=1).max()


# ---------------------------------------------------------------------------------------------------
# Sec. 3.1: a second score for the structured mask (squared Euclidean norm of the group's residual rows).
def test_l2_group_score(oracle):
    rng = np.random.default_rng(6)
    r = (_rand_w(rng, 40, 70) * np.exp(rng.uniform(-2, 2, size=(40, 1)))).astype(np.float32)
    g, n_keep = 4, 3
    kept, score = oracle.select_groups_ex(r, g, n_keep, oracle.SCORE_L2)
    exact_score = [math.fsum(float(v) ** 2 for v in r[j * g:(j + 1) * g].reshape(-1)) for j in range(10)]
    np.testing.assert_allclose(score, exact_score, rtol=1e-14)
    ranked = sorted(range(10), key=lambda j: (-exact_score[j], j))
    np.testing.assert_array_equal(kept, sorted(ranked[:n_keep]))
    # the two scores can disagree: one large entry against many middling ones
    r2 = np.zeros((8, 16), np.float32)
    r2[0, 0] = 1.0            # group 0: max 1, energy 1
    r2[4:8, :] = 0.5          # group 1: max 0.5, energy 16
    assert list(oracle.select_groups_ex(r2, 4, 1, oracle.SCORE_MAXABS)[0]) == [0]
    assert list(oracle.select_groups_ex(r2, 4, 1, oracle.SCORE_L2)[0]) == [1]
    # ties go to the lower index
    r3 = np.tile(np.array([[0.25, -0.5]], np.float32), (12, 1))
    assert list(oracle.select_groups_ex(r3, 4, 2, oracle.SCORE_L2)[0]) == [0, 1]
    # max-abs mode is the pinned selection
    a = oracle.row_absmax(r)
    np.testing.assert_array_equal(oracle.select_groups_ex(r, g, n_keep, oracle.SCORE_MAXABS)[0], oracle.select_groups(a, g, n_keep))


# Sec. 3.1: the unstructured mask.
def test_unstructured_mask(oracle):
    rng = np.random.default_rng(7)
    O, I, bits, K, n_e = 12, 37, 4, 3, 9
    W = _rand_w(rng, O, I)
    e = oracle.expand_ex(W, bits, K, 4, 3, elem_keep=n_e)
    assert list(e.kept_count) == [3, 3, 3]                      # every order keeps every row
    first = oracle.expand_ex(W, bits, 1, 4, 3)
    np.testing.assert_array_equal(e.order_codes(0), first.order_codes(0))     # order 1 is dense
    r = first.residual.copy()
    for k in (1, 2):
        q, s = e.order_codes(k), e.order_scales(k)
        for o in range(O):
            order = sorted(range(I), key=lambda i: (-abs(float(r[o, i])), i))    # independent: a full sort per row
            keep = sorted(order[:n_e])
            assert not np.delete(q[o], keep).any()                               # everything else carries the code 0
            assert s[o] == np.float32(np.abs(r[o]).max()) / np.float32(7)
            for i in range(I):
                if i in keep:
                    c = max(-7, min(7, exact.rne_int(exact.f32(exact.frac(r[o, i]) / exact.frac(s[o])))))
                    assert q[o, i] == c
                    r[o, i] = np.float32(float(exact.f32(exact.frac(r[o, i]) - exact.frac(s[o]) * c)))
    np.testing.assert_array_equal(r.view(np.uint32), e.residual.view(np.uint32))   # pruned entries kept their residual
    # keeping every entry is the plain expansion
    full = oracle.expand_ex(W, bits, K, 4, 3, elem_keep=I)
    plain = oracle.expand_ex(W, bits, K, 4, 3)
    np.testing.assert_array_equal(full.codes, plain.codes)
    # and the masked expansion still converges: each order shrinks the kept entries' error
    assert np.abs(e.residual).max() <= np.abs(first.residual).max()


# ---------------------------------------------------------------------------------------------------
# Sec. 3.2: the activation functions of the ensemble approximation, against the math library.
def test_activation_functions(oracle):
    v = np.array([-30.0, -3.0, -1.0, -1e-3, 0.0, 1e-3, 0.5, 1.0, 3.0, 30.0], np.float32)
    np.testing.assert_array_equal(oracle.activation(v, oracle.ACT_IDENTITY), v)
    np.testing.assert_array_equal(oracle.activation(v, oracle.ACT_RELU), np.maximum(v, 0))
    sig = np.array([1.0 / (1.0 + math.exp(-float(t))) for t in v])
    np.testing.assert_allclose(oracle.activation(v, oracle.ACT_SIGMOID), sig, rtol=1e-6)
    np.testing.assert_allclose(oracle.activation(v, oracle.ACT_SILU), v * sig, rtol=1e-6, atol=1e-12)
    gelu = np.array([0.5 * float(t) * (1.0 + math.erf(float(t) / math.sqrt(2.0))) for t in v])
    np.testing.assert_allclose(oracle.activation(v, oracle.ACT_GELU), gelu, rtol=1e-6, atol=1e-12)
    # closed-form anchors: sigma(0) = 1/2, SiLU(0) = GeLU(0) = 0, large arguments pass through / vanish
    assert oracle.activation(np.zeros(1, np.float32), oracle.ACT_SIGMOID)[0] == 0.5
    assert oracle.activation(np.array([30.0], np.float32), oracle.ACT_GELU)[0] == 30.0
    assert abs(oracle.activation(np.array([-30.0], np.float32), oracle.ACT_SILU)[0]) < 1e-11
    # the ensemble approximation of Sec. 3.2, sigma(a + eps) ~ sigma(a) + sigma(eps), to first order at a smooth point
    a, eps = np.float32(0.7), np.float32(1e-3)
    for kind in (oracle.ACT_SILU, oracle.ACT_GELU):
        lhs = oracle.activation(np.array([a + eps], np.float32), kind)[0]
        rhs = oracle.activation(np.array([a], np.float32), kind)[0] + oracle.activation(np.array([eps], np.float32), kind)[0]
        assert abs(float(lhs) - float(rhs)) < 2e-3
