"""Appendix C (upper bounds U_res / U_sparse) and the choice of (K, gamma, [K_m]) from a budget of bit operations
(Sec. 3.1, App. A, App. H): the library's host functions against the oracle's closed forms, and the closed forms
against what the mathematics fixes -- special cases, a measured error that must stay below the bound on synthetic
layers, NumPy's SVD for the spectral norm, the paper's own example budgets.  No GPU."""
import math

import numpy as np
import pytest

from oracle import pipe_oracle as O
from paper_2311_15806_b200 import binding as B
from paper_2311_15806_b200 import build as pipe_build


@pytest.fixture(scope="module")
def lib():
    pipe_build.build()
    return B.lib()


def test_network_bound_closed_forms(lib):
    # one layer: U = s u; two layers: (s1 u1 + 1)(s1 u1 + s2 u2 + 1) - 1, expanded by hand
    assert O.bound_network([3.0], [0.25]) == pytest.approx(0.75)
    s1, u1, s2, u2 = 2.0, 0.1, 5.0, 0.02
    assert O.bound_network([s1, s2], [u1, u2]) == pytest.approx(s1 * u1 + (s1 * u1 + s2 * u2) + s1 * u1 * (s1 * u1 + s2 * u2))
    # no quantization error, no bound; monotone in every step
    assert O.bound_network([4.0, 7.0, 2.0], [0.0, 0.0, 0.0]) == 0.0
    base = O.bound_network([4.0, 7.0, 2.0], [0.01, 0.02, 0.03])
    assert O.bound_network([4.0, 7.0, 2.0], [0.01, 0.03, 0.03]) > base
    rng = np.random.default_rng(0)
    for L in (1, 2, 5):
        s, u = rng.uniform(0.5, 4, L), rng.uniform(0, 0.1, L)
        assert B.pipe_bound_network(s, u) == pytest.approx(O.bound_network(s, u), rel=1e-14)
    assert B.pipe_bound_network([1.0], [-1.0]) < 0


def test_dense_step_is_lemma_b1(lib):
    for bits, K, lam in [(8, 1, 0.02), (4, 3, 0.5), (2, 8, 1.0), (3, 2, 0.1), (6, 4, 0.3)]:
        want = O.bound_step_dense(bits, K, lam)
        assert want == pytest.approx(lam / 2 / (2 ** (bits - 1) - 1) ** (K - 1))
        assert B.pipe_bound_step_dense(bits, K, lam) == pytest.approx(want, rel=1e-14)
    # the step really bounds the expansion's error (the lemma, on a synthetic layer)
    rng = np.random.default_rng(1)
    W = (rng.standard_normal((32, 48)) * 0.05).astype(np.float32)
    for bits, K in [(4, 2), (3, 3), (8, 2)]:
        e = O.expand_ex(W, bits, K, 4, 8)
        assert np.abs(e.residual).max() <= O.bound_step_dense(bits, K, float(e.order_scales(0).max())) * (1 + 1e-6)


def test_spectral_norm_against_svd(lib):
    rng = np.random.default_rng(2)
    for shape in [(40, 25), (16, 64), (1, 9), (30, 30)]:
        W = rng.standard_normal(shape).astype(np.float32)
        want = np.linalg.svd(W.astype(np.float64), compute_uv=False)[0]
        assert B.pipe_spectral_norm(W, 500, 1e-12) == pytest.approx(want, rel=1e-6)
    assert B.pipe_spectral_norm(np.zeros((3, 4), np.float32)) == 0.0
    # a rank-one matrix: |a| |b|
    a, b = rng.standard_normal(12), rng.standard_normal(7)
    assert B.pipe_spectral_norm(np.outer(a, b).astype(np.float32)) == pytest.approx(np.linalg.norm(a) * np.linalg.norm(b), rel=1e-5)


def test_measured_error_of_a_two_layer_relu_network_stays_below_the_bound(lib):
    """The first theorem of Appendix C on synthetic layers: F(x) = B relu(A x); both layers expanded; the largest
    output error over unit-norm inputs must not exceed U_res built from the spectral norms and the steps."""
    rng = np.random.default_rng(3)
    A = (rng.standard_normal((48, 32)) * 0.2).astype(np.float32)
    Bm = (rng.standard_normal((24, 48)) * 0.2).astype(np.float32)
    X = rng.standard_normal((400, 32))
    X /= np.linalg.norm(X, axis=1, keepdims=True)
    for bits, K, n_keep in [(4, 2, 12), (8, 1, 12), (3, 3, 12), (4, 3, 6)]:
        eA, eB = O.expand_ex(A, bits, K, 4, n_keep), O.expand_ex(Bm, bits, K, 4, min(n_keep, 6))
        AK, BK = A.astype(np.float64) - eA.residual, Bm.astype(np.float64) - eB.residual   # what the expansions represent
        err = np.abs(np.maximum(X @ A.T.astype(np.float64), 0) @ Bm.T.astype(np.float64) - np.maximum(X @ AK.T, 0) @ BK.T).max()
        s = [B.pipe_spectral_norm(A), B.pipe_spectral_norm(Bm)]
        # the theorem's u is RELATIVE (s_{A - A^(K)} <= s_A u_A); a step in the weights' own units gives it through
        # |A - A^(K)|_2 <= sqrt(O I) * max|residual|
        def rel_step(W, e):
            last = np.zeros(W.shape[0], np.float32)
            for k in range(e.K):
                last[e.order_channels(k)] = e.order_scales(k)
            u_abs = B.pipe_bound_step_rows(last)
            assert np.abs(e.residual).max() <= u_abs * (1 + 1e-6)      # half the last step bounds every row
            return math.sqrt(W.size) * u_abs / B.pipe_spectral_norm(W)
        U = B.pipe_bound_network(s, [rel_step(A, eA), rel_step(Bm, eB)])
        assert err <= U
    # a dense expansion: the row-wise step is never above Lemma B.1's
    e = O.expand_ex(A, 4, 3, 4, 12)
    last = e.order_scales(2)[np.argsort(e.order_channels(2))]
    assert B.pipe_bound_step_rows(last) <= B.pipe_bound_step_dense(4, 3, float(e.order_scales(0).max())) * (1 + 1e-6)


SHAPES = [(3, 56, 256, 256, 1), (1, 1, 768, 3072, 1), (1, 1, 11008, 4096, 1), (3, 112, 32, 64, 2)]


@pytest.mark.parametrize("shape", SHAPES)
def test_expansion_choice_from_a_budget(lib, shape):
    d, D, ni, no, s = shape
    full = O.bit_ops_original(d, D, ni, no, s)
    for bits, frac, kmax, gmin, M in [(4, 0.25, 8, 0.25, 2), (2, 0.10, 8, 0.25, 4), (4, 1.0, 16, 0.5, 3), (8, 0.2, 4, 0.25, 1),
                                      (3, 0.15, 8, 0.125, 2)]:
        budget = frac * full
        K, gamma, split = B.pipe_choose_expansion(d, D, ni, no, s, bits, budget, kmax, gmin, M)
        assert (K, split) == O.choose_expansion(d, D, ni, no, s, bits, budget, kmax, gmin, M)[::2]
        assert gamma == pytest.approx(O.choose_expansion(d, D, ni, no, s, bits, budget, kmax, gmin, M)[1], rel=1e-12)
        # what the choice costs stays within the budget, one more order's worth would not (unless capped)
        beta = O.budget_of(K, gamma)
        assert O.bit_ops_expanded(d, D, ni, no, s, bits, beta) <= budget * (1 + 1e-9)
        assert 1 <= K <= kmax and (K == 1 or gamma >= gmin - 1e-9) and gamma <= 1.0
        assert sum(split) == K and len(split) == min(M, K) and split == sorted(split, reverse=True)
    # the paper's own example: a ternary expansion at budget 7 runs at order 8 (App. A), i.e. gamma = 6/7
    rescale = O.bit_ops_expanded(d, D, ni, no, s, 2, 0.0)
    budget7 = O.bit_ops_expanded(d, D, ni, no, s, 2, 7.0)
    K, gamma, _ = B.pipe_choose_expansion(d, D, ni, no, s, 2, budget7, 8, 0.25, 1)
    assert K == 8 and gamma == pytest.approx(6.0 / 7.0)
    # "150 %": order 2 at half density
    K, gamma, _ = B.pipe_choose_expansion(d, D, ni, no, s, 4, O.bit_ops_expanded(d, D, ni, no, s, 4, 1.5), 2, 0.25, 1)
    assert K == 2 and gamma == pytest.approx(0.5)
    # a budget below one order is refused
    with pytest.raises(B.PipeError):
        B.pipe_choose_expansion(d, D, ni, no, s, 4, rescale * 1.0000001, 8, 0.25, 1)
