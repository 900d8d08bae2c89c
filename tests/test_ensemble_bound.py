"""The ensemble approximation on a two-layer ReLU network (Sec. 3.2: sigma(a + eps) ~ sigma(a) + sigma(eps); appendix
"Upper Bound Error", the corollary of the two-layer lemma as printed:
U ~ 1/2 * sum_k ||R_2^(k)|| * sum_{k > K_1} ||R_1^(k)||, spectral norms of the de-quantized orders, ||x|| = 1).

Oracle only, no GPU.  Two ways to read what the LAST layer of a predictor holds are evaluated side by side:
  A  every layer of predictor m holds cluster m only (the reading the library implements: the grouped launch
     gives predictor m its own orders on its own input, and the predictors are added after the last layer);
  B  the appendix's L-layer equations: inner layers as in A, the last layer applies ALL K orders to the sum of
     the predictors' activations.
What the test fixes: both stay below the corollary's U; B is the closer approximation of the full expansion; A's
distance from the full expansion is that of the plain K_1-order expansion to within a few percent, because its
second predictor is a product of two tails."""
import numpy as np
import pytest


def _dense_order(e, k):
    """Order k (0-based) of an expansion as a dense float64 [O, I] matrix s_k * q_k; rows of pruned groups are zero."""
    Wk = np.zeros((e.O, e.I))
    lo = e.row_off(k)
    for j, grp in enumerate(e.kept[k][:e.kept_count[k]]):
        rows = slice(lo + j * e.g, lo + (j + 1) * e.g)
        Wk[grp * e.g:(grp + 1) * e.g] = e.codes[rows].astype(np.float64) * e.scales[rows, None].astype(np.float64)
    return Wk


@pytest.mark.parametrize("bits,K,K1,gamma", [(4, 4, 2, 1.0), (4, 2, 1, 1.0), (8, 2, 1, 1.0), (2, 8, 4, 1.0), (2, 8, 6, 1.0),
                                             (4, 4, 2, 0.5)])
def test_two_layer_ensemble_error_against_the_corollary(oracle, bits, K, K1, gamma):
    rng = np.random.default_rng(100 * bits + 10 * K + K1)
    I, Hd, O, T, g = 128, 256, 64, 128, 8
    W1 = (rng.standard_normal((Hd, I)) / np.sqrt(I)).astype(np.float32)
    W2 = (rng.standard_normal((O, Hd)) / np.sqrt(Hd)).astype(np.float32)
    b1 = (rng.standard_normal(Hd) * 0.1).astype(np.float32)
    b2 = (rng.standard_normal(O) * 0.1).astype(np.float32)
    e1 = oracle.expand(W1, bits, K, g, oracle.keep_groups(Hd // g, gamma))
    e2 = oracle.expand(W2, bits, K, g, oracle.keep_groups(O // g, gamma))
    x = rng.standard_normal((T, I)).astype(np.float32)
    x /= np.linalg.norm(x, axis=1, keepdims=True)
    xq, sx = oracle.quantize_act(x)

    D1 = [_dense_order(e1, k) for k in range(K)]
    D2 = [_dense_order(e2, k) for k in range(K)]
    W2_all, W2_g = sum(D2), sum(D2[:K1])
    W2_h = W2_all - W2_g
    # first layer through the oracle's forward (binary64 sums of the exact integer partials)
    y_all = oracle.forward(e1, xq, sx, bias=b1).y64
    y_g = oracle.forward(e1, xq, sx, 0, K1, bias=b1).y64
    y_h = oracle.forward(e1, xq, sx, K1, K).y64
    np.testing.assert_allclose(y_g + y_h, y_all, rtol=0, atol=1e-12)       # the clusters partition the orders
    relu = lambda v: np.maximum(v, 0)
    full = relu(y_all) @ W2_all.T + b2                                    # F^(K)
    ens_a = relu(y_g) @ W2_g.T + b2 + relu(y_h) @ W2_h.T                  # reading A
    ens_b = (relu(y_g) + relu(y_h)) @ W2_all.T + b2                       # reading B
    trunc = relu(y_g) @ W2_g.T + b2                                       # F^(K_1): the first predictor alone

    err = lambda d: float(np.linalg.norm(d, axis=1).mean())
    U = 0.5 * sum(np.linalg.norm(d, 2) for d in D2) * sum(np.linalg.norm(d, 2) for d in D1[K1:])
    ea, eb, et = err(full - ens_a), err(full - ens_b), err(full - trunc)
    assert eb <= U and ea <= U
    assert eb < ea
    assert abs(ea - et) <= 0.05 * et
    # sigma(a + eps) = sigma(a) + sigma(eps) wherever a and eps are both non-negative or the sum stays
    # negative with eps negative (the approximation of Sec. 3.2 is an identity there), so B's error lives on the other rows only
    same = (np.sign(y_g) == np.sign(y_h)) | (y_h == 0)
    assert np.allclose((relu(y_g) + relu(y_h))[same], relu(y_all)[same], atol=1e-12)
